// Attention backward (Algorithm 1 of the paper, Section 4.1) for sm_100a.
//
// Three kernels per call:
//   bwd_preprocess_kernel : delta = rowsum(dO * O); writes -delta and -LSE/scale as fp16
//                           (hi, lo) pairs, zeroes the fp32 dQ accumulator, records
//                           max |delta|, max ||dO_row||^2 and max ||V_row||^2 (together they bound |dS|)
//   bwd_main_kernel       : per (batch, kv head, key tile j): loop over the group's
//                           query heads and the visible query tiles i, recompute
//                           P^T from LSE, and run the five tile contractions on
//                           tcgen05 tensor cores with tensor-memory accumulators
//   bwd_finalize_kernel   : dQ fp32 accumulator -> fp16
//
// Loop order differs from Algorithm 1 (which is query-outer and reduces dK/dV partials
// across workers): here a CTA owns one key/value tile, keeps dK_j and dV_j resident in
// tensor memory for the whole loop, and the cross-CTA reduction falls on dQ instead.
//
// The main kernel is persistent (one CTA per SM claims work items, heavy ones first, from a counter)
// and warp specialised: 16 warps in four warpgroups, so that each group can resize its share of the
// register file (the control group hands most of its registers to the other three):
//   warp 0       TMA producer (one thread): K_j, V_j once; then a two-stage ring of Q_i and a
//                single-buffered dO_i; the warp also owns the tensor-memory allocation
//   warp 1       tensor-core issuer (one thread); warps 2-3 only fill up the control group
//   warps 4-11   softmax / dS warps: warps 4-7 take query columns 0-63 of a tile pair,
//                warps 8-11 columns 64-127; each thread owns one key row
//   warps 12-15  dQ reduction (tensor memory -> shared memory -> bulk add.f32 into the fp32
//                accumulator: linear 8 KB pieces at D = 128, swizzled boxes through a tensor map at
//                D = 64) and the per-item dK/dV epilogue
// Transposed scores are used (S^T = K Q^T, dP^T = V dO^T) so that P^T, written back to
// tensor memory as fp16, is directly the A operand of dV += P^T dO; dS^T is written both to
// tensor memory (A operand of dK += dS^T Q) and to shared memory (operand of the dQ product).
// The row terms -LSE_i/scale and -delta_i are added inside the S^T and dP^T products by one
// extra 16-element contraction step whose operands are (256, 1, 0...) and the (hi, lo, 0...)
// split of the term, so the softmax warps never touch LSE or delta.
//
// Instantiations of the main kernel: fp16 or bf16 operands; a variant that splits a group's query
// heads over several work items (few, heavy items) and sums dK/dV in fp32 in the workspace; and a
// variant that loads the probability tiles a forward pass saved (Section 4.1's own forward state,
// written by lt_attn_save_p) instead of recomputing them.
#include <mutex>
#include <stddef.h>
#include <stdio.h>

#include "lt_common.cuh"
#include "lt_host.h"

namespace lt {

constexpr int kTileRows = 128;             // rows of a query tile and of a key/value tile
constexpr int kBoxBytesBwd = 128 * 128;    // one swizzled tile of 128 rows x 64 fp16
constexpr float kLog2e = 1.4426950408889634f;

// wait codes recorded in the status block when a bounded wait gives up
enum {
    kWaitKV = 201, kWaitStageEmpty = 202, kWaitStageFull = 203, kWaitSFull = 204, kWaitPReady = 205,
    kWaitDpFull = 206, kWaitDsReady = 207, kWaitDsFree = 208, kWaitDqFull = 209, kWaitDqEmpty = 210,
    kWaitDkvFull = 211, kWaitDoFull = 212, kWaitDoEmpty = 213, kWaitAccFree = 214,
    kWaitItem = 200, kBadSmemAlign = 220
};

// ----------------------------------------------------------------------------- preprocess
// One half-warp (D = 128) or quarter-warp (D = 64) per row, 16-byte loads of dO and O; each
// warp works on kPreUnroll groups of rows at a time so that enough loads are in flight to
// keep HBM busy.
constexpr int kPreUnroll = 4;

template <int D, bool kBf16>
__global__ void __launch_bounds__(256, 3)  // three blocks per multiprocessor keep enough loads in flight
bwd_preprocess_kernel(const __half *__restrict__ dO, const __half *__restrict__ O, const float *__restrict__ lse,
                      uint4 *__restrict__ delta_ext, uint4 *__restrict__ lse_ext, float *__restrict__ dq_acc,
                      long long n_rows, int S, int S_pad, int Hq, lt_tensor_strides do_st, lt_tensor_strides o_st,
                      int plain, float inv_scale, unsigned int *status, float4 *__restrict__ kv_acc,
                      long long kv_acc_vec4, const __half *__restrict__ V, long long v_rows, int Hkv,
                      lt_tensor_strides v_st, int v_plain) {
    // `n_rows` counts rows of the padded row space (every head rounded up to S_pad rows), the
    // indexing of delta_ext, lse_ext and dq_acc; padding rows get zeros everywhere.
    grid_launch_dependents();  // the main kernel sets itself up while this kernel's last blocks run
    // fp32 dK/dV sums (only when key tiles are split over several work items): zero them
    for (long long v = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; v < kv_acc_vec4;
         v += static_cast<long long>(gridDim.x) * blockDim.x)
        kv_acc[v] = make_float4(0.f, 0.f, 0.f, 0.f);
    constexpr int kLanesPerRow = D / 8;
    constexpr int kRowsPerWarp = 32 / kLanesPerRow;
    constexpr int kRowsPerTrip = kRowsPerWarp * kPreUnroll;
    const int lane = threadIdx.x & 31;
    const int sub = lane % kLanesPerRow;
    const long long warp_global = (static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5;
    const long long n_warps = (static_cast<long long>(gridDim.x) * blockDim.x) >> 5;
    float max_abs_delta = 0.f, max_norm2 = 0.f;
    for (long long row0 = warp_global * kRowsPerTrip; row0 < n_rows; row0 += n_warps * kRowsPerTrip) {
        uint4 a[kPreUnroll], b[kPreUnroll];
        float l[kPreUnroll];
#pragma unroll
        for (int u = 0; u < kPreUnroll; ++u) {
            const long long row = row0 + u * kRowsPerWarp + lane / kLanesPerRow;
            a[u] = b[u] = make_uint4(0u, 0u, 0u, 0u);
            l[u] = 0.f;
            // rows of dO, O and LSE behind padded row `row` (`plain`: contiguous tensors and no padding,
            // so all three are row `row` itself)
            long long src_do = row * D, src_o = row * D, src_lse = row;
            bool valid = row < n_rows;
            if (!plain && valid) {
                const int bh = static_cast<int>(row / S_pad);
                const int s_in = static_cast<int>(row - static_cast<long long>(bh) * S_pad);
                const int bb = bh / Hq, hh = bh - bb * Hq;
                valid = s_in < S;
                src_do = bb * do_st.batch + hh * do_st.head + s_in * do_st.row;
                src_o = bb * o_st.batch + hh * o_st.head + s_in * o_st.row;
                src_lse = static_cast<long long>(bh) * S + s_in;
            }
            if (valid) {
                a[u] = __ldcs(reinterpret_cast<const uint4 *>(dO + src_do) + sub);
                b[u] = __ldcs(reinterpret_cast<const uint4 *>(O + src_o) + sub);
                if (sub == 0 && lse) l[u] = __ldg(lse + src_lse);  // (no LSE in the saved-P variant)
            }
            if (row < n_rows) {
                // the zero fill does not depend on the loads: issue it while they are in flight
                float4 *z = reinterpret_cast<float4 *>(dq_acc + row * D) + sub * 2;
                z[0] = make_float4(0.f, 0.f, 0.f, 0.f);
                z[1] = make_float4(0.f, 0.f, 0.f, 0.f);
            }
        }
#pragma unroll
        for (int u = 0; u < kPreUnroll; ++u) {
            const long long row = row0 + u * kRowsPerWarp + lane / kLanesPerRow;
            const uint32_t *ah = reinterpret_cast<const uint32_t *>(&a[u]);
            const uint32_t *bh = reinterpret_cast<const uint32_t *>(&b[u]);
            float acc = 0.f, n2 = 0.f;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float2 x = unpack2<kBf16>(ah[e]);
                const float2 y = unpack2<kBf16>(bh[e]);
                acc = fmaf(x.x, y.x, acc);
                acc = fmaf(x.y, y.y, acc);
                n2 = fmaf(x.x, x.x, n2);
                n2 = fmaf(x.y, x.y, n2);
            }
#pragma unroll
            for (int off = kLanesPerRow / 2; off > 0; off >>= 1) {
                acc += __shfl_xor_sync(0xffffffffu, acc, off);
                n2 += __shfl_xor_sync(0xffffffffu, n2, off);
            }
            if (row < n_rows) {
                if (sub == 0) {
                    // operand rows of the main kernel's extra contraction step: 256*hi + lo = value
                    delta_ext[row] = split_ext<kBf16>(-acc);
                    lse_ext[row] = split_ext<kBf16>(-l[u] * inv_scale);
                }
                max_abs_delta = fmaxf(max_abs_delta, fabsf(acc));
                max_norm2 = fmaxf(max_norm2, n2);
            }
        }
    }
    // largest squared row norm of V (rows of the logical [B,Hkv,S]): with the two maxima above it bounds
    // |dS|, from which the main kernel picks the power of two that dS carries into fp16
    // (kept as bit patterns: non-negative floats order like them, with inf above every finite value and
    // NaN above inf, so non-finite inputs saturate the bound)
    unsigned int max_v2 = 0u;
    for (long long row0 = warp_global * kRowsPerTrip; row0 < v_rows; row0 += n_warps * kRowsPerTrip) {
        uint4 a[kPreUnroll];
#pragma unroll
        for (int u = 0; u < kPreUnroll; ++u) {
            const long long row = row0 + u * kRowsPerWarp + lane / kLanesPerRow;
            a[u] = make_uint4(0u, 0u, 0u, 0u);
            if (row < v_rows) {
                long long src = row * D;
                if (!v_plain) {
                    const int bg = static_cast<int>(row / S);
                    const int s_in = static_cast<int>(row - static_cast<long long>(bg) * S);
                    const int bb = bg / Hkv, gg = bg - bb * Hkv;
                    src = bb * v_st.batch + gg * v_st.head + s_in * v_st.row;
                }
                a[u] = __ldg(reinterpret_cast<const uint4 *>(V + src) + sub);  // (the main kernel reads V again)
            }
        }
#pragma unroll
        for (int u = 0; u < kPreUnroll; ++u) {
            const uint32_t *ah = reinterpret_cast<const uint32_t *>(&a[u]);
            float n2 = 0.f;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float2 x = unpack2<kBf16>(ah[e]);
                n2 = fmaf(x.x, x.x, n2);
                n2 = fmaf(x.y, x.y, n2);
            }
#pragma unroll
            for (int off = kLanesPerRow / 2; off > 0; off >>= 1) n2 += __shfl_xor_sync(0xffffffffu, n2, off);
            max_v2 = max(max_v2, __float_as_uint(n2) & 0x7fffffffu);
        }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        max_abs_delta = fmaxf(max_abs_delta, __shfl_xor_sync(0xffffffffu, max_abs_delta, off));
        max_norm2 = fmaxf(max_norm2, __shfl_xor_sync(0xffffffffu, max_norm2, off));
        max_v2 = max(max_v2, __shfl_xor_sync(0xffffffffu, max_v2, off));
    }
    // one set of atomics per block, and only when it would raise the stored maximum: thousands of
    // atomics on the same words would otherwise queue up behind one another in L2
    __shared__ float block_max[3][8];
    if (lane == 0) {
        block_max[0][threadIdx.x >> 5] = max_abs_delta;
        block_max[1][threadIdx.x >> 5] = max_norm2;
        block_max[2][threadIdx.x >> 5] = __uint_as_float(max_v2);
    }
    __syncthreads();
    if (threadIdx.x < 3) {
        unsigned int m = 0u;
#pragma unroll
        for (int w = 0; w < 8; ++w) m = max(m, __float_as_uint(block_max[threadIdx.x][w]) & 0x7fffffffu);
        unsigned int *word = status + (threadIdx.x == 0 ? kStatusWordMaxAbsDelta
                                       : threadIdx.x == 1 ? kStatusWordMaxDoNorm2 : kStatusWordMaxVNorm2);
        if (m > *reinterpret_cast<volatile unsigned int *>(word)) atomicMax(word, m);
    }
}

// ----------------------------------------------------------------------------- finalize
template <bool kBf16>
__global__ void __launch_bounds__(256)
bwd_finalize_kernel(const float *__restrict__ dq_acc, __half *__restrict__ dQ, long long n_vec8, int vec_per_head,
                    int vec_per_padded_head, int vec_per_row, int Hq, lt_tensor_strides dq_st, int plain) {
    // n_vec8 groups of eight output elements, numbered over the logical [B,Hq,S,D]; the accumulator
    // is indexed in the padded row space (`plain`: contiguous dQ and no padding, so both are group v)
    grid_dependency_wait();  // launched while the main kernel drains: its reductions must have landed
    const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
    for (long long v = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; v < n_vec8; v += stride) {
        long long src = v, dst = v * 8;
        if (!plain) {
            const int bh = static_cast<int>(v / vec_per_head);
            const int rem = static_cast<int>(v - static_cast<long long>(bh) * vec_per_head);
            const int s_in = rem / vec_per_row, c = rem - s_in * vec_per_row;
            const int bb = bh / Hq, hh = bh - bb * Hq;
            src = static_cast<long long>(bh) * vec_per_padded_head + rem;
            dst = bb * dq_st.batch + hh * dq_st.head + s_in * dq_st.row + c * 8;
        }
        const float4 a = __ldcs(reinterpret_cast<const float4 *>(dq_acc) + 2 * src);
        const float4 b = __ldcs(reinterpret_cast<const float4 *>(dq_acc) + 2 * src + 1);
        uint4 o;
        o.x = pack2<kBf16>(a.x, a.y);
        o.y = pack2<kBf16>(a.z, a.w);
        o.z = pack2<kBf16>(b.x, b.y);
        o.w = pack2<kBf16>(b.z, b.w);
        *reinterpret_cast<uint4 *>(dQ + dst) = o;
    }
}

// fp32 dK / dV sums [B,Hkv,S_pad,D] -> 16-bit outputs (only when key tiles were split over work items)
template <bool kBf16>
__global__ void __launch_bounds__(256)
bwd_finalize_kv_kernel(const float *__restrict__ dk_acc, const float *__restrict__ dv_acc, __half *__restrict__ dK,
                       __half *__restrict__ dV, long long n_vec8, int vec_per_head, int vec_per_padded_head,
                       int vec_per_row, int Hkv, lt_tensor_strides dk_st, lt_tensor_strides dv_st) {
    grid_dependency_wait();  // every share of the main kernel must have landed
    const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
    for (long long v = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; v < 2 * n_vec8; v += stride) {
        const bool second = v >= n_vec8;
        const long long u = second ? v - n_vec8 : v;
        const int bh = static_cast<int>(u / vec_per_head);
        const int rem = static_cast<int>(u - static_cast<long long>(bh) * vec_per_head);
        const int s_in = rem / vec_per_row, c = rem - s_in * vec_per_row;
        const int bb = bh / Hkv, hh = bh - bb * Hkv;
        const long long src = static_cast<long long>(bh) * vec_per_padded_head + rem;
        const lt_tensor_strides &st = second ? dv_st : dk_st;
        const long long dst = bb * st.batch + hh * st.head + s_in * st.row + c * 8;
        const float *acc = second ? dv_acc : dk_acc;
        const float4 a = __ldcs(reinterpret_cast<const float4 *>(acc) + 2 * src);
        const float4 b = __ldcs(reinterpret_cast<const float4 *>(acc) + 2 * src + 1);
        uint4 o;
        o.x = pack2<kBf16>(a.x, a.y);
        o.y = pack2<kBf16>(a.z, a.w);
        o.z = pack2<kBf16>(b.x, b.y);
        o.w = pack2<kBf16>(b.z, b.w);
        *reinterpret_cast<uint4 *>((second ? dV : dK) + dst) = o;
    }
}

// ----------------------------------------------------------------------------- optional cycle trace
// Built only with -DLT_BWD_TRACE (development aid): per-role cycle totals, summed over all CTAs.
// Slot = 16 * role + (wait code - 200); slot 16 * role + 15 = the role's whole loop.
enum { kRoleProducer = 0, kRoleMma = 1, kRoleCompute = 2, kRoleReduce = 3 };
#ifdef LT_BWD_TRACE
__device__ unsigned long long g_bwd_trace[80];
struct Trace {
    unsigned int acc[16];
    unsigned int t0;
    __device__ __forceinline__ void start() {
        t0 = static_cast<unsigned int>(clock());
#pragma unroll
        for (int i = 0; i < 16; ++i) acc[i] = 0;
    }
    __device__ __forceinline__ void flush(int role) {
        acc[15] = static_cast<unsigned int>(clock()) - t0;
        if ((threadIdx.x & 31) == 0) {
#pragma unroll
            for (int i = 0; i < 16; ++i)
                if (acc[i]) atomicAdd(&g_bwd_trace[16 * role + i], static_cast<unsigned long long>(acc[i]));
        }
    }
};
#define LT_TRACE_BEGIN() Trace trace_; trace_.start()
#define LT_TRACE_MARK(var) const unsigned int var = static_cast<unsigned int>(clock())
#define LT_TRACE_SINCE(slot, var) trace_.acc[slot] += static_cast<unsigned int>(clock()) - var
#define LT_TRACE_END(role) trace_.flush(role)
#define LT_WAIT(bar, parity, code) traced_wait(trace_, bar, parity, abort_flag, p.status, code)
__device__ __forceinline__ bool traced_wait(Trace &tr, uint64_t *bar, uint32_t parity, volatile int *abort_flag,
                                            unsigned int *status, int code) {
    const unsigned int t0 = static_cast<unsigned int>(clock());
    const bool r = mbar_wait(bar, parity, abort_flag, status, code);
    tr.acc[code - 200] += static_cast<unsigned int>(clock()) - t0;
    return r;
}
#else
#define LT_TRACE_BEGIN()
#define LT_TRACE_MARK(var)
#define LT_TRACE_SINCE(slot, var)
#define LT_TRACE_END(role)
#define LT_WAIT(bar, parity, code) mbar_wait(bar, parity, abort_flag, p.status, code)
#endif
// the same wait by every lane of a warp, with the outcome voted (warp-uniform)
#define LT_WAIT_ALL(bar, parity, code) __all_sync(0xffffffffu, LT_WAIT(bar, parity, code))

// Built only with -DLT_BWD_TIMELINE=<cta> (development aid): clock stamps of that CTA's first 256 iterations.
#ifdef LT_BWD_TIMELINE
__device__ long long g_bwd_timeline[20 * 256];  // [event][iteration]; events are listed in paper_2606_10415_b200/timeline.py
#define LT_TL(cond, ev, iter)                                                                        \
    do {                                                                                             \
        if ((cond) && blockIdx.x == LT_BWD_TIMELINE && (iter) < 256) g_bwd_timeline[(ev) * 256 + (iter)] = clock64(); \
    } while (0)
#else
#define LT_TL(cond, ev, iter) do {} while (0)
#endif

// ----------------------------------------------------------------------------- main kernel
constexpr int kQStages = 2;   // Q_i ring; dO_i is single-buffered (it is dead once dV has been issued)
constexpr int kBwdThreads = 512;  // 16 warps; 128 registers per thread at launch
constexpr int kComputeWarp0 = 4, kNumComputeWarps = 8;
constexpr int kReduceWarp0 = 12, kNumReduceWarps = 4;
// registers per thread once the warpgroups have resized their shares (the SM has 64 K)
constexpr int kRegsAtLaunch = 65536 / kBwdThreads;
constexpr int kRegsControl = 56, kRegsCompute = 160, kRegsReduce = 136;
static_assert(128 * kRegsControl + kNumComputeWarps * 32 * kRegsCompute + kNumReduceWarps * 32 * kRegsReduce <= 65536,
              "register shares exceed the register file");
constexpr int kDqStageBufs = 3, kDqStageRows = 16;
constexpr int kExtBytes = 2048;            // 128 rows x 16 bytes: one operand of the extra contraction step
constexpr float kPScaleLog2Max = 14.f;     // P is kept as P * 2^c with c <= 14 so that fp16(P') <= 16384
constexpr int kBarReduceWarps = 1;  // named barrier id
constexpr int kItemRing = 4;  // roles are never more than two items apart
constexpr double kL2BatchBytes = 80.0e6;  // working set of one batch of work items (L2 holds 126 MB)

template <int D>
struct BwdSmem {
    static constexpr int kBoxes = D / 64;
    static constexpr int kTile = kBoxes * kBoxBytesBwd;
    uint8_t k[kTile];
    uint8_t v[kTile];
    uint8_t q[kQStages][kTile];
    uint8_t d_o[kTile];
    uint8_t ds[2 * kBoxBytesBwd];      // dS^T: rows = key index, 128 query columns in two swizzled tiles
    // operands of the extra contraction step that subtracts LSE/scale from S and delta from dP
    uint8_t ext_ones[kExtBytes];       // rows (256, 1, 0...): goes with K_j and with V_j
    uint8_t ext_q[kQStages][kExtBytes];// rows (hi, lo, 0...) of -LSE/scale for the stage's query tile
    uint8_t ext_do[kExtBytes];         // rows (hi, lo, 0...) of -delta
    uint8_t ext_zero[kExtBytes];       // contraction elements 8-15 of all of the above
    // staging of the dQ partial for bulk reduction into global memory (D = 128 only):
    // each buffer holds 16 accumulator rows (16 query rows x 128 floats)
    // (D = 64: two buffers of a whole partial, 128 query rows x 64 floats, each as two swizzled boxes of 32 columns)
    float dq_stage[D == 128 ? kDqStageBufs : 2][D == 128 ? kDqStageRows * 128 : kTileRows * 64];
    // per work item: K/V landed; dK/dV accumulators complete; accumulators read out
    uint64_t bar_kv, bar_dkv_full, bar_acc_free;
    // work items are claimed from a global counter by the producer and published to the other roles
    uint64_t bar_item[kItemRing];
    int item_ring[kItemRing];
    // per (query head, query tile) iteration
    uint64_t bar_q_full[kQStages], bar_q_empty[kQStages], bar_do_full, bar_do_empty;
    uint64_t bar_s_full, bar_p_ready, bar_dp_full, bar_ds_ready, bar_ds_free, bar_dq_full, bar_dq_empty;
    uint32_t tmem_base;
    int abort_flag;
};

static_assert(sizeof(BwdSmem<128>) <= 232448, "main kernel shared memory exceeds the 227 KB per-block limit");

struct BwdParams {
    const uint4 *lse_ext;    // per query row: fp16 (hi, lo, 0 x 6) with 256*hi + lo = -LSE / scale
    const uint4 *delta_ext;  // per query row: fp16 (hi, lo, 0 x 6) with 256*hi + lo = -delta
    float *dq_acc;
    __half *dK;
    __half *dV;
    unsigned int *status;
    int B, Hq, Hkv, S, S_pad, causal;  // S_pad: S rounded up to whole 128-row tiles
    // (batch, kv head) units per L2-sized batch of work items.  In the variant that splits a group of
    // query heads over several items the word also carries, above bit 16, the items per (unit, key
    // tile) and, above bit 24, the query heads per item; dK and dV then point at the fp32 sums
    // [B,Hkv,S_pad,D] of the parts.  (The structure keeps its size: the main kernel's register
    // allocation is sensitive to it.)
    int units_per_batch;
    float scale;
    lt_tensor_strides dk_st, dv_st;  // element strides of dK and dV
};

// One work item = key tile j of (batch b, kv head g).  Items are numbered so that the heavy
// ones (small j under a causal mask) come first; CTA c takes items c, c + gridDim.x, ...
struct BwdItem {
    int j, b, g, i_first, tiles_per_head, n_iter;
    int h_first;  // first query head of the group this item covers (0 unless the group is split)
};
template <bool kSplit>
__device__ __forceinline__ BwdItem bwd_item(const BwdParams &p, int item) {
    BwdItem w;
    const int parts = kSplit ? ((p.units_per_batch >> 16) & 0xFF) : 1;
    const int units_per_batch = kSplit ? (p.units_per_batch & 0xFFFF) : p.units_per_batch;
    const int heads_per_item = kSplit ? ((p.units_per_batch >> 24) & 0xFF) : 0;
    const int n_tiles = (p.S + kTileRows - 1) / kTileRows;  // the last tile may be ragged
    const int n_bg = p.B * p.Hkv;
    // Items are numbered batch of (batch, kv head) units by batch; inside a batch key tile by key tile
    // (heavy tiles first), all units of the batch per key tile.  A batch is sized so that everything its
    // items touch (K, V, the group's Q and dO, the fp32 dQ rows) stays in L2 while the CTAs work
    // through it; with one batch this is the plain heavy-first order.
    const int batch = item / (units_per_batch * n_tiles * parts);
    const int first_unit = batch * units_per_batch;
    const int units = min(units_per_batch, n_bg - first_unit);
    // A group of query heads may be split into `parts` items per key tile (shapes with few, heavy
    // items); the parts of one key tile are neighbours in the numbering.
    const int within = item - first_unit * n_tiles * parts;
    w.j = within / (units * parts);
    const int rem = within - w.j * units * parts;
    const int unit_local = rem / parts;
    const int part = rem - unit_local * parts;
    const int bg = first_unit + unit_local;
    w.b = bg / p.Hkv;
    w.g = bg - w.b * p.Hkv;
    w.i_first = p.causal ? w.j : 0;
    w.tiles_per_head = n_tiles - w.i_first;
    if constexpr (kSplit) {
        w.h_first = part * heads_per_item;
        w.n_iter = min(heads_per_item, p.Hq / p.Hkv - w.h_first) * w.tiles_per_head;
    } else {
        w.h_first = 0;
        w.n_iter = (p.Hq / p.Hkv) * w.tiles_per_head;  // flattened (query head of the group, query tile) loop
    }
    return w;
}
// Iteration n of an item -> its query tile: batch, query head, first row inside the head, and the tile's first row in the padded row space of the workspace arrays
// (every head rounded up to whole tiles, so tiles never straddle heads).
struct BwdQTile {
    int b, h, s0;
    long long padded_row0;
};
__device__ __forceinline__ BwdQTile bwd_q_tile(const BwdParams &p, const BwdItem &w, int n) {
    const int hh = n / w.tiles_per_head;
    const int i = w.i_first + (n - hh * w.tiles_per_head);
    BwdQTile q;
    q.b = w.b;
    q.h = w.g * (p.Hq / p.Hkv) + w.h_first + hh;
    q.s0 = i * kTileRows;
    q.padded_row0 = (static_cast<long long>(w.b) * p.Hq + q.h) * p.S_pad + q.s0;
    return q;
}

// The saved P^T tile (128 keys x 128 queries, fp16, 32 KB) of key tile w.j and query tile qt.
__device__ __forceinline__ const __half *saved_p_tile(const BwdParams &p, const BwdItem &w, const BwdQTile &qt) {
    const long long n_tiles = p.S_pad / kTileRows;
    const long long tile = ((static_cast<long long>(qt.b) * p.Hq + qt.h) * n_tiles + w.j) * n_tiles + qt.s0 / kTileRows;
    return reinterpret_cast<const __half *>(p.lse_ext) + tile * (kTileRows * kTileRows);
}

// The exponent c of the power of two that P carries (P' = P * 2^c, c <= 14), and with it dS, so that
// dS' uses fp16's normal range without overflow when it is rounded: chosen from a bound on
// |dS| <= |dP| + |delta| <= max ||dO_row|| * max ||V_row|| + max |delta| over the whole call (the
// three maxima come from the preprocess kernel).  dV and dQ / dK undo the factor exactly in their
// epilogues.  Every thread that needs c computes it once per CTA from the status block.
__device__ __forceinline__ int bwd_p_scale_log2(const unsigned int *status) {
    const float do2 = __uint_as_float(__ldcg(status + kStatusWordMaxDoNorm2));
    const float v2 = __uint_as_float(__ldcg(status + kStatusWordMaxVNorm2));
    const float dmax = __uint_as_float(__ldcg(status + kStatusWordMaxAbsDelta));
    const float bound = sqrtf(do2) * sqrtf(v2) + dmax;
    if (!(bound < 3.0e38f)) return -14;                           // inf/NaN inputs: outputs are non-finite anyway
    if (!(bound > 1e-30f)) return static_cast<int>(kPScaleLog2Max);  // all-zero dO: any factor works
    return min(static_cast<int>(kPScaleLog2Max), max(-14, ilogbf(32768.f / bound)));
}

// kSavedP: the variant that loads the probability tiles a forward pass saved (lt_attn_save_p's store)
// instead of recomputing them.  It issues no S product; the producer asks for each P^T tile to be
// brought into L2 one iteration ahead and every softmax thread reads its own 128 bytes of the tile
// straight into registers.  BwdParams::lse_ext, which this variant does not need, carries the
// store's address (the parameter block keeps its size).
template <int D, bool kBf16, bool kSplit, bool kSavedP = false>
__global__ void __launch_bounds__(kBwdThreads, 1)
bwd_main_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_do,
                const BwdParams p, const __grid_constant__ CUtensorMap map_dq) {
    // map_dq (D = 64 only): the fp32 dQ accumulator as rows of 64 floats, boxes of 128 rows x 32 columns
    using Smem = BwdSmem<D>;
    constexpr int kBoxes = D / 64;
    constexpr uint32_t kTileBytes = kBoxes * kBoxBytesBwd;
    constexpr uint32_t kTmemCols = 512;
    constexpr uint32_t kColS = 0, kColdP = 128, kColdV = 256, kColdK = 384;

    extern __shared__ __align__(1024) uint8_t smem_raw[];
    Smem &sm = *reinterpret_cast<Smem *>(smem_raw);
#ifdef LT_BWD_TRACE
    const long long trace_cta_t0 = clock64();
#endif
    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;
    const int n_items = (p.S_pad / kTileRows) * p.B * p.Hkv * (kSplit ? ((p.units_per_batch >> 16) & 0xFF) : 1);

    // the swizzled tiles need 1024-byte alignment; the shared window is expected to give it
    const bool smem_ok = (smem_u32(smem_raw) & 1023u) == 0u;
    if (tid == 0) {
        sm.abort_flag = smem_ok ? 0 : 1;
        if (!smem_ok) atomicCAS(p.status + kStatusWordTimeout, 0u, static_cast<unsigned int>(kBadSmemAlign));
        mbar_init(&sm.bar_kv, 1);
        mbar_init(&sm.bar_dkv_full, 1);
        mbar_init(&sm.bar_acc_free, kNumReduceWarps);
        for (int r = 0; r < kItemRing; ++r) mbar_init(&sm.bar_item[r], 1);
        for (int s = 0; s < kQStages; ++s) {
            mbar_init(&sm.bar_q_full[s], 1);
            mbar_init(&sm.bar_q_empty[s], 1);
        }
        mbar_init(&sm.bar_do_full, 1);
        mbar_init(&sm.bar_do_empty, 1);
        mbar_init(&sm.bar_s_full, 1);
        mbar_init(&sm.bar_p_ready, kNumComputeWarps);
        mbar_init(&sm.bar_dp_full, 1);
        mbar_init(&sm.bar_ds_ready, kNumComputeWarps);
        mbar_init(&sm.bar_ds_free, 1);
        mbar_init(&sm.bar_dq_full, 1);
        mbar_init(&sm.bar_dq_empty, kNumReduceWarps);
        mbar_fence_init();
        tma_prefetch_desc(&map_q);
        tma_prefetch_desc(&map_k);
        tma_prefetch_desc(&map_v);
        tma_prefetch_desc(&map_do);
    }
    if (warp == 0) {
        tmem_alloc(&sm.tmem_base, kTmemCols);
        tmem_relinquish();
    }
    if (warp == 1) {
        // constant operands of the extra contraction step
        const uint2 mult = ext_multipliers<kBf16>();
        for (int r = lane; r < kTileRows; r += 32) {
            reinterpret_cast<uint4 *>(sm.ext_ones)[r] = make_uint4(mult.x, mult.y, 0u, 0u);
            reinterpret_cast<uint4 *>(sm.ext_zero)[r] = make_uint4(0u, 0u, 0u, 0u);
        }
        fence_proxy_async_smem();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    // everything above ran while the preprocess kernel was finishing; its results (row operands, zeroed
    // accumulator, running maxima, item counter) are read only from here on
    grid_dependency_wait();
    const uint32_t tmem = sm.tmem_base;
    volatile int *abort_flag = &sm.abort_flag;
#ifdef LT_BWD_TRACE
    const long long trace_prologue_end = clock64();
    int trace_iters = 0;
#endif

    // Every role walks the same list of work items and keeps its own running iteration count
    // `it` (over all items): each per-iteration barrier completes once per iteration, so its
    // phase parity is a function of `it`; the per-item barriers use the item count `ic`.
    if (warp < kComputeWarp0) {
        // ================================================================= control group
        warpgroup_regs_set<kRegsControl, kRegsAtLaunch>();
        if (warp == 0) {
            // ================================================================= TMA producer
            if (lane == 0 && smem_ok) {
                LT_TRACE_BEGIN();
                bool ok = true;
                int it = 0, ic = 0;
                int last_q = -1, last_do = -1, kv_loads = 0;  // for the cleanup after an abandoned wait
                // claim the next unclaimed item (heavy ones have the low numbers) and publish it to the
                // other roles; -1 tells everybody that the list is exhausted
                auto claim = [&](int slot_ic) -> int {
                    const unsigned int v = atomicAdd(p.status + kStatusWordItemCounter, 1u);
                    const int item = v < static_cast<unsigned int>(n_items) ? static_cast<int>(v) : -1;
                    sm.item_ring[slot_ic % kItemRing] = item;
                    mbar_arrive(&sm.bar_item[slot_ic % kItemRing]);
                    return item;
                };
                int item = claim(0);
                while (item >= 0 && ok) {
                    const BwdItem w = bwd_item<kSplit>(p, item);
                    int next_item = -1;
                    for (int n = 0; n < w.n_iter && ok; ++n, ++it) {
                        const int s = it & 1, k = it >> 1;
                        const BwdQTile qt = bwd_q_tile(p, w, n);
                        if (k >= 1 && !(ok = LT_WAIT(&sm.bar_q_empty[s], (k - 1) & 1, kWaitStageEmpty))) break;
                        mbar_arrive_expect_tx(&sm.bar_q_full[s], kSavedP ? kTileBytes : kTileBytes + kExtBytes);
#pragma unroll
                        for (int x = 0; x < kBoxes; ++x)
                            tma_load_4d(sm.q[s] + x * kBoxBytesBwd, &map_q, &sm.bar_q_full[s], x * 64, qt.s0, qt.h, qt.b);
                        if constexpr (kSavedP)
                            bulk_prefetch_l2(saved_p_tile(p, w, qt), kTileRows * kTileRows * 2);
                        else
                            bulk_load_1d(sm.ext_q[s], p.lse_ext + qt.padded_row0, kExtBytes, &sm.bar_q_full[s]);
                        last_q = it;
                        if (it >= 1 && !(ok = LT_WAIT(&sm.bar_do_empty, (it - 1) & 1, kWaitDoEmpty))) break;
                        mbar_arrive_expect_tx(&sm.bar_do_full, kTileBytes + kExtBytes);
#pragma unroll
                        for (int x = 0; x < kBoxes; ++x)
                            tma_load_4d(sm.d_o + x * kBoxBytesBwd, &map_do, &sm.bar_do_full, x * 64, qt.s0, qt.h, qt.b);
                        bulk_load_1d(sm.ext_do, p.delta_ext + qt.padded_row0, kExtBytes, &sm.bar_do_full);
                        last_do = it;
                        if (n == 0) {
                            // K_j and V_j follow the first query tile: they may only be overwritten once every
                            // product of the previous item has completed
                            if (ic >= 1 && !(ok = LT_WAIT(&sm.bar_dkv_full, (ic - 1) & 1, kWaitDkvFull))) break;
                            mbar_arrive_expect_tx(&sm.bar_kv, 2 * kTileBytes);
#pragma unroll
                            for (int x = 0; x < kBoxes; ++x) {
                                tma_load_4d(sm.k + x * kBoxBytesBwd, &map_k, &sm.bar_kv, x * 64, w.j * kTileRows, w.g, w.b);
                                tma_load_4d(sm.v + x * kBoxBytesBwd, &map_v, &sm.bar_kv, x * 64, w.j * kTileRows, w.g, w.b);
                            }
                            ++kv_loads;
                        }
                        if (n == w.n_iter - 1) {
                            // with the last query tile of this item on its way, claim the next item and ask for
                            // its K/V tiles to be brought into L2 while this item finishes
                            next_item = claim(ic + 1);
                            if (next_item >= 0) {
                                const BwdItem wn = bwd_item<kSplit>(p, next_item);
#pragma unroll
                                for (int x = 0; x < kBoxes; ++x) {
                                    tma_prefetch_l2_4d(&map_k, x * 64, wn.j * kTileRows, wn.g, wn.b);
                                    tma_prefetch_l2_4d(&map_v, x * 64, wn.j * kTileRows, wn.g, wn.b);
                                }
                            }
                        }
                    }
                    item = next_item;
                    ++ic;
                }
                LT_TRACE_END(kRoleProducer);
                if (*abort_flag) {
                    // abandoned: give this CTA's own copies a bounded time to land before shared memory is released
                    if (kv_loads > 0)
                        for (int t = 0; t < (1 << 16) && !mbar_try_wait(&sm.bar_kv, (kv_loads - 1) & 1); ++t) {}
                    for (int n = max(0, last_q - 1); n <= last_q; ++n)
                        for (int t = 0; t < (1 << 16) && !mbar_try_wait(&sm.bar_q_full[n & 1], (n >> 1) & 1); ++t) {}
                    if (last_do >= 0)
                        for (int t = 0; t < (1 << 16) && !mbar_try_wait(&sm.bar_do_full, last_do & 1); ++t) {}
                }
            }
            __syncwarp();
        } else if (warp == 1) {
            // ================================================================= tensor-core issuer
            // The whole warp walks the loop, so that loop counters, wait results (voted) and descriptor arithmetic are
            // warp-uniform; one elected lane issues the products and commits.
            if (smem_ok) {
                const bool leader = elect_one();
                LT_TRACE_BEGIN();
                // Every operand descriptor is a compile-time constant (built from the operand's offset inside
                // the shared window) plus the window's base in the address field (bits 0-13, units of 16
                // bytes; shared memory stays below 256 KB, so the sum never carries out of the field).  The
                // issuing thread spends one 64-bit add per descriptor, so the tensor pipe, not this thread,
                // sets the pace.  The base is re-read through window_base() once per tile pair: otherwise the
                // compiler keeps all ~80 sums of an iteration in registers across the loop, and the control
                // group could not hand most of its registers to the other warpgroups.
                const uint32_t base16 = smem_u32(smem_raw) >> 4;
                auto window_base = [&]() -> uint64_t {
                    uint32_t v;
                    asm volatile("mov.u32 %0, %1;" : "=r"(v) : "r"(base16));
                    return static_cast<uint64_t>(v);
                };
                constexpr uint32_t oK = offsetof(Smem, k), oV = offsetof(Smem, v), oQ = offsetof(Smem, q);
                constexpr uint32_t oDo = offsetof(Smem, d_o), oDs = offsetof(Smem, ds), oZero = offsetof(Smem, ext_zero);
                constexpr uint32_t oOnes = offsetof(Smem, ext_ones), oExtQ = offsetof(Smem, ext_q), oExtDo = offsetof(Smem, ext_do);
                constexpr uint64_t dK_k = desc_kmajor(oK), dV_k = desc_kmajor(oV);
                constexpr uint64_t dK_mn = desc_mnmajor(oK, kBoxBytesBwd);
                constexpr uint64_t ddS_mn = desc_mnmajor(oDs, kBoxBytesBwd);
                constexpr uint64_t ddO_k = desc_kmajor(oDo), ddO_mn = desc_mnmajor(oDo, kBoxBytesBwd);
                constexpr uint64_t dQ_k0 = desc_kmajor(oQ), dQ_mn0 = desc_mnmajor(oQ, kBoxBytesBwd);
                constexpr uint64_t kQStageStep = static_cast<uint64_t>(Smem::kTile) >> 4;  // next Q stage
                constexpr uint64_t desc_ones = desc_kmajor_noswz(oOnes, oZero - oOnes, 128);
                constexpr uint64_t desc_ext_do = desc_kmajor_noswz(oExtDo, oZero - oExtDo, 128);
                constexpr uint64_t desc_ext_q0 = desc_kmajor_noswz(oExtQ, oZero - oExtQ, 128);
                constexpr uint64_t desc_ext_q1 = desc_kmajor_noswz(oExtQ + kExtBytes, oZero - oExtQ - kExtBytes, 128);
                // address-field increments of contraction step kk: within a contraction-contiguous tile
                // (32 bytes per step, next 64-column tile after four steps) and within a row-contracted
                // tile (16 rows of 128 bytes per step)
                constexpr auto koff = [](int kk) -> uint64_t { return static_cast<uint64_t>((kk >> 2) * (kBoxBytesBwd >> 4) + (kk & 3) * 2); };
                constexpr auto roff = [](int kk) -> uint64_t { return static_cast<uint64_t>(kk * (2048 >> 4)); };
                constexpr uint32_t idesc_s = make_idesc(128, 128, false, false, kBf16);
                constexpr uint32_t idesc_dv = make_idesc(128, D, false, true, kBf16);
                constexpr uint32_t idesc_dq = make_idesc(128, D == 128 ? 128 : D, true, true, kBf16);
                auto issue_s = [&](int t) {  // S^T = K_j Q_i^T - LSE_i / scale, for running iteration t
                    if (!leader) return;
                    const uint64_t wb = window_base();
                    const uint64_t dQ_k = wb + (t & 1) * kQStageStep;
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk)
                        umma_ss(tmem + kColS, wb + (dK_k + koff(kk)), dQ_k + (dQ_k0 + koff(kk)), idesc_s, kk > 0);
                    umma_ss(tmem + kColS, wb + desc_ones, wb + ((t & 1) ? desc_ext_q1 : desc_ext_q0), idesc_s, 1);
                    umma_commit(&sm.bar_s_full);
                };
                bool ok = true;
                int it = 0, ic = 0;
                for (;; ++ic) {
                    if (!(ok = LT_WAIT_ALL(&sm.bar_item[ic % kItemRing], (ic / kItemRing) & 1, kWaitItem))) break;
                    const int item = sm.item_ring[ic % kItemRing];
                    if (item < 0) break;
                    const BwdItem w = bwd_item<kSplit>(p, item);
                    ok = LT_WAIT_ALL(&sm.bar_kv, ic & 1, kWaitKV) &&
                         LT_WAIT_ALL(&sm.bar_q_full[it & 1], (it >> 1) & 1, kWaitStageFull);
                    if (!ok) break;
                    tc_fence_after_sync();
                    LT_TL(leader, 14, it);
                    if constexpr (!kSavedP) issue_s(it);
                    for (int n = 0; n < w.n_iter && ok; ++n, ++it) {
                        const int s = it & 1;
                        const uint64_t wb = window_base();
                        const uint64_t dQ_mn = wb + s * kQStageStep;
                        // dO_i and the -delta rows have landed: both dP and dV read them
                        if (!(ok = LT_WAIT_ALL(&sm.bar_do_full, it & 1, kWaitDoFull))) break;
                        // dP^T = V_j dO_i^T - delta_i   (its columns held the previous dQ partial until the
                        //                                reduce warps drained it)
                        auto issue_dp = [&]() {
                            if (!leader) return;
#pragma unroll
                            for (int kk = 0; kk < D / 16; ++kk)
                                umma_ss(tmem + kColdP, wb + (dV_k + koff(kk)), wb + (ddO_k + koff(kk)), idesc_s, kk > 0);
                            umma_ss(tmem + kColdP, wb + desc_ones, wb + desc_ext_do, idesc_s, 1);
#ifdef LT_BWD_GIVEUP_TEST
                            // test build only: the hand-off of running iteration LT_BWD_GIVEUP_TEST is dropped, so
                            // the waits downstream of it run out and the kernel has to leave through its give-up path
                            if (it != LT_BWD_GIVEUP_TEST)
#endif
                            umma_commit(&sm.bar_dp_full);
                        };
                        // dV_j += P'^T dO_i   (A = P'^T from tensor memory; query columns 0-63 sit at columns
                        //                      0-31, query columns 64-127 at columns 64-95 of the S region)
                        auto issue_dv = [&]() {
                            if (!leader) return;
#pragma unroll
                            for (int kk = 0; kk < 8; ++kk)
                                umma_ts(tmem + kColdV, tmem + kColS + (kk >> 2) * 64 + (kk & 3) * 8, wb + (ddO_mn + roff(kk)),
                                        idesc_dv, (n > 0) | (kk > 0));
                        };
                        LT_TL(leader, 0, it);
                        if (it > 0 && !(ok = LT_WAIT_ALL(&sm.bar_dq_empty, (it - 1) & 1, kWaitDqEmpty))) break;
                        tc_fence_after_sync();
                        LT_TL(leader, 1, it);
                        issue_dp();
                        LT_TL(leader, 2, it);
                        if (!(ok = LT_WAIT_ALL(&sm.bar_p_ready, it & 1, kWaitPReady))) break;
                        LT_TL(leader, 3, it);
                        // the first product of an item overwrites accumulators the previous item's epilogue reads
                        if (n == 0 && ic > 0 && !(ok = LT_WAIT_ALL(&sm.bar_acc_free, (ic - 1) & 1, kWaitAccFree))) break;
                        tc_fence_after_sync();
                        issue_dv();
                        if (leader) umma_commit(&sm.bar_do_empty);
                        // the next S^T overwrites P'^T; the tensor pipe executes in issue order
                        if (n + 1 < w.n_iter) {
                            if (!(ok = LT_WAIT_ALL(&sm.bar_q_full[(it + 1) & 1], ((it + 1) >> 1) & 1, kWaitStageFull))) break;
                            if constexpr (!kSavedP) issue_s(it + 1);
                        }
                        LT_TL(leader, 4, it);
                        if (!(ok = LT_WAIT_ALL(&sm.bar_ds_ready, it & 1, kWaitDsReady))) break;
                        tc_fence_after_sync();
                        LT_TL(leader, 5, it);
                        // dK_j += dS'^T Q_i   (A = dS'^T from tensor memory, stored like P'^T: query columns
                        //                       0-63 at columns 0-31 and 64-127 at columns 64-95 of the dP region)
                        if (leader) {
#pragma unroll
                            for (int kk = 0; kk < 8; ++kk)
                                umma_ts(tmem + kColdK, tmem + kColdP + (kk >> 2) * 64 + (kk & 3) * 8, dQ_mn + (dQ_mn0 + roff(kk)), idesc_dv,
                                        (n > 0) | (kk > 0));
                            umma_commit(&sm.bar_q_empty[s]);
                        }
                        // dQ_i partial (contraction over key rows); it overwrites the dP columns, which is safe
                        // after dK because the tensor pipe executes in issue order.  For D = 128 it is
                        // produced transposed, dQ^T = K_j^T dS^T (lanes = head dim, columns = query rows), so
                        // that the reduction moves whole accumulator rows; for D = 64 as dQ = dS K_j.
                        if (leader) {
#pragma unroll
                            for (int kk = 0; kk < 8; ++kk) {
                                if constexpr (D == 128)
                                    umma_ss(tmem + kColdP, wb + (dK_mn + roff(kk)), wb + (ddS_mn + roff(kk)), idesc_dq, kk > 0);
                                else
                                    umma_ss(tmem + kColdP, wb + (ddS_mn + roff(kk)), wb + (dK_mn + roff(kk)), idesc_dq, kk > 0);
                            }
                            umma_commit(&sm.bar_dq_full);
                            umma_commit(&sm.bar_ds_free);
                        }
                        LT_TL(leader, 6, it);
                    }
                    if (!ok) break;
                    if (leader) umma_commit(&sm.bar_dkv_full);
                }
                LT_TRACE_END(kRoleMma);
            }
            __syncwarp();
        }
    } else if (warp < kReduceWarp0) {
        // ================================================================= softmax / dS warps
        warpgroup_regs_set<kRegsCompute, kRegsAtLaunch>();
        const int quad = warp & 3;                           // tensor-memory lane quadrant
        const int half_sel = (warp - kComputeWarp0) >> 2;    // 0: query columns 0-63, 1: 64-127
        const int row = quad * 32 + lane;                    // key row inside the tile
        const uint32_t lane_base = static_cast<uint32_t>(quad * 32) << 16;
        const uint32_t cbase = half_sel * 64;
        const float scale_log2 = p.scale * kLog2e;
        uint8_t *ds_tile = sm.ds + half_sel * kBoxBytesBwd;
        uint32_t pv[64];  // bits of this thread's 64 fp32 values of P' = P * 2^c for the current tile pair
        const float p_scale_log2 = static_cast<float>(bwd_p_scale_log2(p.status));
        bool ok = smem_ok;
        int it = 0, ic = 0;
        LT_TRACE_BEGIN();

        // saved-P variant: this thread's 64 saved probabilities of the current tile pair (ph) and of the
        // next one (pn, in flight while dS of the current pair is formed), as packed fp16 pairs
        uint32_t ph[32], pn[32];
        auto load_saved_p = [&](const BwdItem &w, int n, uint32_t *dst) {
            // the store keeps a tile as sixteen blocks of eight query columns, each [128 keys][8 queries]:
            // the 32 lanes of a warp (consecutive key rows) read 512 contiguous bytes per load
            const uint4 *src = reinterpret_cast<const uint4 *>(saved_p_tile(p, w, bwd_q_tile(p, w, n))) + (cbase / 8) * kTileRows + row;
#pragma unroll
            for (int v = 0; v < 8; ++v) {
                const uint4 u = ld_nc_v4(src + v * kTileRows);
                dst[4 * v] = u.x; dst[4 * v + 1] = u.y; dst[4 * v + 2] = u.z; dst[4 * v + 3] = u.w;
            }
        };
        auto compute_p = [&](const BwdItem &w, int n, int t) -> bool {
            if constexpr (kSavedP) {
                // P'^T of the previous pair must have been read by its dV product before it is replaced
                if (t > 0 && !LT_WAIT(&sm.bar_do_empty, (t - 1) & 1, kWaitDoEmpty)) return false;
                tc_fence_after_sync();
                const uint32_t mult = pack_half2(exp2f(p_scale_log2), exp2f(p_scale_log2));  // 2^c <= 2^14
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    uint32_t out[16];
#pragma unroll
                    for (int e = 0; e < 16; ++e) out[e] = hmul2_bits(ph[c * 16 + e], mult);
                    tmem_st16(tmem + lane_base + kColS + cbase + c * 16, out);
                }
                tmem_wait_st();
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(&sm.bar_p_ready);
                return true;
            }
            if (!LT_WAIT(&sm.bar_s_full, t & 1, kWaitSFull)) return false;
            tc_fence_after_sync();
            LT_TL(tid == kComputeWarp0 * 32, 7, t);
            LT_TRACE_MARK(tp0);
            const int hh = n / w.tiles_per_head;
            const bool diag = p.causal && (w.i_first + (n - hh * w.tiles_per_head) == w.j);
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                // (one load at a time: asking for both halves before the first is used measured 2 % slower)
                uint32_t sv[32];
                tmem_ld32(tmem + lane_base + kColS + cbase + c * 32, sv);
                tmem_wait_ld();
                // P' = exp2(scale*log2e * (K.Q - LSE/scale) + c)
#pragma unroll
                for (int e = 0; e < 32; ++e)
                    pv[c * 32 + e] = __float_as_uint(fast_exp2(fmaf(__uint_as_float(sv[e]), scale_log2, p_scale_log2)));
            }
            if (diag) {  // key row is hidden from query column q when row > q
#pragma unroll
                for (int e = 0; e < 64; ++e)
                    if (row > static_cast<int>(cbase) + e) pv[e] = 0u;
            }
            if (w.j * kTileRows + row >= p.S) {
                // a key row past the end of the sequence (ragged last tile): its zero-filled K row has
                // score 0, which LSE does not bound, so its P is not a probability; hide it
#pragma unroll
                for (int e = 0; e < 64; ++e) pv[e] = 0u;
            }
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                uint32_t out[16];
#pragma unroll
                for (int e = 0; e < 16; ++e)
                    out[e] = pack2<kBf16>(__uint_as_float(pv[c * 32 + 2 * e]), __uint_as_float(pv[c * 32 + 2 * e + 1]));
                // in place: these columns lie inside the 64 columns this thread has just read
                tmem_st16(tmem + lane_base + kColS + cbase + c * 16, out);
            }
            tmem_wait_st();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.bar_p_ready);
            LT_TL(tid == kComputeWarp0 * 32, 8, t);
            LT_TRACE_SINCE(12, tp0);
            return true;
        };

        for (;; ++ic) {
            if (!ok || !LT_WAIT(&sm.bar_item[ic % kItemRing], (ic / kItemRing) & 1, kWaitItem)) break;
            const int item = sm.item_ring[ic % kItemRing];
            if (item < 0) break;
            const BwdItem w = bwd_item<kSplit>(p, item);
            if constexpr (kSavedP) load_saved_p(w, 0, ph);
            ok = compute_p(w, 0, it);
            for (int n = 0; n < w.n_iter && ok; ++n, ++it) {
                if constexpr (kSavedP)
                    if (n + 1 < w.n_iter) load_saved_p(w, n + 1, pn);
                if (!(ok = LT_WAIT(&sm.bar_dp_full, it & 1, kWaitDpFull))) break;
                tc_fence_after_sync();
                LT_TL(tid == kComputeWarp0 * 32, 9, it);
                // the previous dS^T tile must have been consumed by the dQ product before it is overwritten
                if (it > 0 && !(ok = LT_WAIT(&sm.bar_ds_free, (it - 1) & 1, kWaitDsFree))) break;
                LT_TRACE_MARK(td0);
                const float saved_mult = kSavedP ? exp2f(p_scale_log2) : 0.f;
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    uint32_t dp[32];
                    tmem_ld32(tmem + lane_base + kColdP + cbase + c * 32, dp);
                    tmem_wait_ld();
                    // dS' = P' * (dP - delta); the subtraction happened inside the tensor-core product.
                    // The fp16 result goes to shared memory (32 query columns = four 16-byte chunks of row
                    // `row` in this half's tile; operand of the dQ product) and, in place, to tensor
                    // memory (operand of dK).
                    uint32_t o[16];
#pragma unroll
                    for (int e = 0; e < 16; ++e) {
                        if constexpr (kSavedP) {
                            const float2 f = unpack2<false>(ph[c * 16 + e]);
                            o[e] = pack2<kBf16>(f.x * saved_mult * __uint_as_float(dp[2 * e]),
                                                f.y * saved_mult * __uint_as_float(dp[2 * e + 1]));
                        } else {
                            o[e] = pack2<kBf16>(__uint_as_float(pv[c * 32 + 2 * e]) * __uint_as_float(dp[2 * e]),
                                                __uint_as_float(pv[c * 32 + 2 * e + 1]) * __uint_as_float(dp[2 * e + 1]));
                        }
                    }
#pragma unroll
                    for (int v4 = 0; v4 < 4; ++v4)
                        *reinterpret_cast<uint4 *>(ds_tile + swz128_offset(row, c * 32 + v4 * 8)) =
                            make_uint4(o[4 * v4], o[4 * v4 + 1], o[4 * v4 + 2], o[4 * v4 + 3]);
                    // these 16 columns lie inside the columns this thread has already read
                    tmem_st16(tmem + lane_base + kColdP + cbase + c * 16, o);
                }
                tmem_wait_st();
                LT_TRACE_SINCE(13, td0);
                fence_proxy_async_smem();
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(&sm.bar_ds_ready);
                LT_TL(tid == kComputeWarp0 * 32, 10, it);
                LT_TRACE_SINCE(14, td0);
                if constexpr (kSavedP) {
#pragma unroll
                    for (int e = 0; e < 32; ++e) ph[e] = pn[e];
                }
                if (n + 1 < w.n_iter) ok = compute_p(w, n + 1, it + 1);
            }

        }
        LT_TRACE_END(kRoleCompute);
    } else {
        // ================================================================= dQ reduction warps
        warpgroup_regs_set<kRegsReduce, kRegsAtLaunch>();
        const int quad = warp & 3;
        // P carried the factor 2^c through dS into the accumulators; the epilogues take it out again (exact)
        const float inv_p_scale = exp2f(-static_cast<float>(bwd_p_scale_log2(p.status)));
        const float dq_mult = p.scale * inv_p_scale;
        bool ok = smem_ok;
        int it = 0, ic = 0;
        uint32_t gq = 0;  // running number of the sixteen-row groups staged so far (D = 128)
        LT_TRACE_BEGIN();
        for (;; ++ic) {
            // the four reduction warps share named barriers (D = 128), so after every wait they vote
            // and leave together
            ok = ok && LT_WAIT(&sm.bar_item[ic % kItemRing], (ic / kItemRing) & 1, kWaitItem);
            ok = named_barrier_and(kBarReduceWarps, kNumReduceWarps * 32, ok);
            if (!ok) break;
            const int item = sm.item_ring[ic % kItemRing];
            if (item < 0) break;
            const BwdItem w = bwd_item<kSplit>(p, item);
            for (int n = 0; n < w.n_iter; ++n, ++it) {
                ok = LT_WAIT(&sm.bar_dq_full, it & 1, kWaitDqFull);
                // The four reduction warps share named barriers below, so they leave the loop together.  The
                // staging buffers form a ring that runs on across tile pairs (running group number gq): at
                // most the last two reductions of the previous pair are still reading their buffers here,
                // the buffer the first group of this pair goes to is free.
                if constexpr (D == 128)
                    if (warp == kReduceWarp0 && lane == 0) bulk_wait_group_read<2>();
                ok = named_barrier_and(kBarReduceWarps, kNumReduceWarps * 32, ok);
                if (!ok) break;
                tc_fence_after_sync();
                LT_TL(tid == kReduceWarp0 * 32, 11, it);
                LT_TRACE_MARK(tr0);
                float *dq_tile = p.dq_acc + bwd_q_tile(p, w, n).padded_row0 * D;
                if constexpr (D == 128) {
                    // dQ^T: this thread holds head-dim element d = 32*quad + lane of all 128 query rows.
                    // Sixteen query rows at a time are scaled, staged in shared memory exactly as they lie
                    // in the accumulator (16 rows x 128 floats, contiguous) and added to it by one bulk
                    // reduction; three staging buffers keep the copies in flight.
                    const int d_idx = quad * 32 + lane;
                    const uint32_t taddr = tmem + (static_cast<uint32_t>(quad * 32) << 16) + kColdP;
                    const bool elected = (warp == kReduceWarp0) && (lane == 0);
                    auto store_rows = [&](int k, const uint32_t *r) {  // r: 16 values, query rows 16k .. 16k+15
                        float *buf = sm.dq_stage[(gq + k) % kDqStageBufs];
#pragma unroll
                        for (int e = 0; e < kDqStageRows; ++e) buf[e * 128 + d_idx] = __uint_as_float(r[e]) * dq_mult;
                    };
                    auto add_rows = [&](int k) {
                        bulk_reduce_add_f32(dq_tile + k * kDqStageRows * 128, sm.dq_stage[(gq + k) % kDqStageBufs],
                                            kDqStageRows * 128 * sizeof(float));
                        bulk_commit_group();
                    };
                    // Seven eighths of the partial are read, one group of rows is parked in shared memory to make
                    // room for the last eighth, and the dP columns are released before any reduction of this
                    // pair is issued.
                    uint32_t r0a[16], r0b[16], r1[32], r2[32], r3[16];
                    tmem_ld16(taddr, r0a);
                    tmem_ld16(taddr + 16, r0b);
                    tmem_ld32(taddr + 32, r1);
                    tmem_ld32(taddr + 64, r2);
                    tmem_ld16(taddr + 96, r3);
                    tmem_wait_ld();
                    store_rows(0, r0a);
                    tmem_ld16(taddr + 112, r0a);
                    tmem_wait_ld();
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&sm.bar_dq_empty);
                    LT_TL(tid == kReduceWarp0 * 32, 12, it);
                    LT_TRACE_SINCE(12, tr0);
                    fence_proxy_async_smem();
                    // the buffer where group 1 goes was read by the last reduction but one of the previous pair
                    if (elected) bulk_wait_group_read<1>();
                    named_barrier_sync(kBarReduceWarps, kNumReduceWarps * 32);
                    if (elected) add_rows(0);
                    // groups 1..7 rotate through the three buffers: before group k is issued, the bulk
                    // reduction of group k-2 has finished reading, which frees the buffer of group k+1
                    auto stage_rows = [&](int k, const uint32_t *r) {
                        store_rows(k, r);
                        fence_proxy_async_smem();
                        if (elected) bulk_wait_group_read<1>();
                        named_barrier_sync(kBarReduceWarps, kNumReduceWarps * 32);
                        if (elected) add_rows(k);
                    };
                    stage_rows(1, r0b);
                    stage_rows(2, r1);
                    stage_rows(3, r1 + 16);
                    stage_rows(4, r2);
                    stage_rows(5, r2 + 16);
                    stage_rows(6, r3);
                    stage_rows(7, r0a);
                    gq += 8;
                } else {
                    // D = 64: dQ partial with lanes = query rows.  A thread holds the 64 floats of one query row.
                    // The partial is scaled and staged in shared memory as two boxes of 128 rows x 32 floats with
                    // the 128-byte swizzle (rows 128 bytes apart: the swizzle spreads a warp's 16-byte stores over
                    // all banks), and two tiled reductions add the boxes to the accumulator; two staging buffers.
                    const int q_row = quad * 32 + lane;
                    const uint32_t taddr = tmem + (static_cast<uint32_t>(quad * 32) << 16) + kColdP;
                    const bool elected = (warp == kReduceWarp0) && (lane == 0);
                    uint32_t r[2][32];
                    tmem_ld32(taddr, r[0]);
                    tmem_ld32(taddr + 32, r[1]);
                    tmem_wait_ld();
                    // the whole partial is in registers: the dP columns may be overwritten
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&sm.bar_dq_empty);
                    LT_TRACE_SINCE(12, tr0);
                    // the buffer of this tile was last read by the reductions issued two tiles ago
                    if (elected) bulk_wait_group_read<1>();
                    named_barrier_sync(kBarReduceWarps, kNumReduceWarps * 32);
                    uint8_t *buf = reinterpret_cast<uint8_t *>(sm.dq_stage[it & 1]);
#pragma unroll
                    for (int bx = 0; bx < 2; ++bx)
#pragma unroll
                        for (int c = 0; c < 8; ++c)
                            *reinterpret_cast<float4 *>(buf + bx * (kTileRows * 128) + q_row * 128 + ((c ^ (q_row & 7)) << 4)) =
                                make_float4(__uint_as_float(r[bx][4 * c]) * dq_mult, __uint_as_float(r[bx][4 * c + 1]) * dq_mult,
                                            __uint_as_float(r[bx][4 * c + 2]) * dq_mult, __uint_as_float(r[bx][4 * c + 3]) * dq_mult);
                    fence_proxy_async_smem();
                    named_barrier_sync(kBarReduceWarps, kNumReduceWarps * 32);
                    if (elected) {
                        const int y = static_cast<int>(bwd_q_tile(p, w, n).padded_row0);
                        tma_reduce_add_2d(&map_dq, buf, 0, y);
                        tma_reduce_add_2d(&map_dq, buf + kTileRows * 128, 32, y);
                        bulk_commit_group();
                    }
                }
                LT_TL(tid == kReduceWarp0 * 32, 13, it);
                LT_TRACE_SINCE(13, tr0);
            }
            if (!ok) break;
            // item epilogue (these warps are idle while the pipeline of the next item fills):
            // dK_j and dV_j leave tensor memory as fp16; thread = key row
            ok = LT_WAIT(&sm.bar_dkv_full, ic & 1, kWaitDkvFull);
            ok = named_barrier_and(kBarReduceWarps, kNumReduceWarps * 32, ok);
            if (!ok) break;
            tc_fence_after_sync();
            {
                const int row = quad * 32 + lane;
                const uint32_t lane_base = static_cast<uint32_t>(quad * 32) << 16;
#pragma unroll
                for (int which = 0; which < 2; ++which) {
                    const float mult = which == 0 ? dq_mult : inv_p_scale;
                    const uint32_t col0 = which == 0 ? kColdK : kColdV;
                    const int s_row = w.j * kTileRows + row;  // rows past S are never stored
                    const lt_tensor_strides &st = which == 0 ? p.dk_st : p.dv_st;
                    __half *dst = (which == 0 ? p.dK : p.dV) + w.b * st.batch + w.g * st.head + s_row * st.row;
#pragma unroll
                    for (int c = 0; c < D / 32; ++c) {
                        uint32_t r[32];
                        tmem_ld32(tmem + lane_base + col0 + c * 32, r);
                        tmem_wait_ld();
                        if (which == 1 && c == D / 32 - 1) {
                            // both accumulators have been read: the next item may overwrite them
                            tc_fence_before_sync();
                            __syncwarp();
                            if (lane == 0) mbar_arrive(&sm.bar_acc_free);
                            LT_TL(tid == kReduceWarp0 * 32, 15, it);
                        }
                        if constexpr (kSplit) {
                            // the group's heads are spread over several items: add this item's share to
                            // the fp32 sums; a separate pass rounds them once all shares are in
                            float *acc = reinterpret_cast<float *>(which == 0 ? p.dK : p.dV) +
                                         ((static_cast<long long>(w.b) * p.Hkv + w.g) * p.S_pad + s_row) * D + c * 32;
                            if (s_row < p.S) {
#pragma unroll
                                for (int v4 = 0; v4 < 8; ++v4)
                                    red_add_v4(acc + 4 * v4, __uint_as_float(r[4 * v4 + 0]) * mult,
                                               __uint_as_float(r[4 * v4 + 1]) * mult, __uint_as_float(r[4 * v4 + 2]) * mult,
                                               __uint_as_float(r[4 * v4 + 3]) * mult);
                            }
                            continue;
                        }
#pragma unroll
                        for (int v8 = 0; v8 < 4; ++v8) {
                            uint4 o;
                            o.x = pack2<kBf16>(__uint_as_float(r[8 * v8 + 0]) * mult, __uint_as_float(r[8 * v8 + 1]) * mult);
                            o.y = pack2<kBf16>(__uint_as_float(r[8 * v8 + 2]) * mult, __uint_as_float(r[8 * v8 + 3]) * mult);
                            o.z = pack2<kBf16>(__uint_as_float(r[8 * v8 + 4]) * mult, __uint_as_float(r[8 * v8 + 5]) * mult);
                            o.w = pack2<kBf16>(__uint_as_float(r[8 * v8 + 6]) * mult, __uint_as_float(r[8 * v8 + 7]) * mult);
                            if (s_row < p.S) reinterpret_cast<uint4 *>(dst + c * 32)[v8] = o;
                        }
                    }
                }
            }
        }
        // shared memory must stay valid until the bulk reductions have read it
        bulk_wait_group_all();
        LT_TRACE_END(kRoleReduce);
#ifdef LT_BWD_TRACE
        trace_iters = it;
#endif
    }

#ifdef LT_BWD_TRACE
    const long long trace_teardown_begin = clock64();
#endif
    grid_launch_dependents();  // the dQ conversion kernel may be scheduled while the last CTAs finish
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, kTmemCols);
#ifdef LT_BWD_TRACE
    if (tid == 0) {
        atomicAdd(&g_bwd_trace[64 + 3], static_cast<unsigned long long>(clock64() - trace_cta_t0));
        atomicAdd(&g_bwd_trace[64 + 1], 1ull);
        atomicAdd(&g_bwd_trace[64 + 0], static_cast<unsigned long long>(trace_prologue_end - trace_cta_t0));
        atomicAdd(&g_bwd_trace[64 + 4], static_cast<unsigned long long>(trace_teardown_begin - trace_prologue_end));
    }
    if (tid == kReduceWarp0 * 32) atomicAdd(&g_bwd_trace[64 + 2], static_cast<unsigned long long>(trace_iters));
#endif
}

#ifdef LT_BWD_TIMELINE
extern "C" int lt_dbg_bwd_timeline(long long *out) {  // out == NULL: clear the stamps
    if (!out) {
        void *sym = nullptr;
        if (cudaGetSymbolAddress(&sym, lt::g_bwd_timeline) != cudaSuccess) return LT_ERR_CUDA;
        return cudaMemset(sym, 0, sizeof(lt::g_bwd_timeline)) == cudaSuccess ? LT_OK : LT_ERR_CUDA;
    }
    return cudaMemcpyFromSymbol(out, lt::g_bwd_timeline, sizeof(lt::g_bwd_timeline)) == cudaSuccess ? LT_OK : LT_ERR_CUDA;
}
#endif
#ifdef LT_BWD_TRACE
extern "C" int lt_dbg_bwd_trace(unsigned long long *out, int reset) {
    if (out && cudaMemcpyFromSymbol(out, g_bwd_trace, sizeof(g_bwd_trace)) != cudaSuccess) return LT_ERR_CUDA;
    if (reset) {
        static unsigned long long zeros[80];
        if (cudaMemcpyToSymbol(g_bwd_trace, zeros, sizeof(zeros)) != cudaSuccess) return LT_ERR_CUDA;
    }
    return LT_OK;
}
#endif

// Query heads of a group per work item.  A (batch, kv head, key tile) item normally covers the whole
// group (dK_j, dV_j of all its heads accumulate in one CTA's tensor memory).  Shapes that would give
// the 148 SMs only a few, heavy items get the group split over several items instead; their shares of
// dK_j, dV_j are then summed in fp32 in the workspace and rounded by a small extra kernel.
// Multiprocessors of the current device (148 on a B200; that figure is also the answer when the query fails,
// so that the sizes derived from it never depend on an error path).
static int sm_count() {
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
        return 148;
    return sms;
}
static int heads_per_item(int B, int Hq, int Hkv, int S, int D, int causal) {
    const int sms = sm_count();
    const long long split_below_items = sms + sms / 2;  // split when there are fewer than 1.5 whole-group items per SM
    const long long split_target_items = 2 * sms;       // and then aim at two items per SM (every item pays a pipeline fill)
    const long long split_min_iterations = 20 * sms;    // problems below this are launch-bound anyway
    const int G = Hq / Hkv;
    const long long n_tiles = padded_rows(S) / kTileRows;
    const long long n_base = static_cast<long long>(B) * Hkv * n_tiles;
    const long long iters = static_cast<long long>(B) * Hq * (causal ? n_tiles * (n_tiles + 1) / 2 : n_tiles * n_tiles);
    if (G == 1 || iters < split_min_iterations) return G;
    if (n_base < split_below_items) {
        const long long split = (split_target_items + n_base - 1) / n_base;
        const int hs = static_cast<int>(split < G ? split : G);
        return (G + hs - 1) / hs;
    }
    // Enough whole-group items to fill the SMs, but too few to form L2-sized batches (a batch needs two items per
    // SM) while the working set is more than four times the L2: the accumulator rows of the heads in flight would be
    // fetched and written back again and again.  Two items per key tile make room for batches.  Measured, whole
    // against split, ms per call: LLaMA-2-70B layer with B = 2 1.78 / 1.69 (3.6 -> 1.45 GB of DRAM traffic), the
    // same at S = 8192 with B = 1 3.38 / 3.02, 32 / 4 heads at S = 16384 6.06 / 5.76.  Smaller working sets lose
    // more to the second pipeline fill and the fp32 epilogue than they gain: 32 / 8 heads at S = 8192 (2.4 L2s)
    // 1.52 / 1.59, the same with B = 2 at S = 4096 0.86 / 0.89, the Qwen2.5-32B layer (1.4 L2s) 0.53 / 0.56.
    const double unit_bytes = static_cast<double>(padded_rows(S)) * D * (2.0 * 2 + G * (2.0 * 2 + 4));
    const double working_set = unit_bytes * B * Hkv;
    if (n_base < 4LL * sms && working_set > 4.0 * 126.0e6) return (G + 1) / 2;
    return G;
}

template <int D, bool kBf16>
static int launch_bwd(const lt_half *Q, const lt_half *K, const lt_half *V, const lt_half *O, const lt_half *dO,
                      const float *LSE, lt_half *dQ, lt_half *dK, lt_half *dV, const lt_attn_layout &lay, int B,
                      int Hq, int Hkv, int S, int causal, float scale, void *workspace, cudaStream_t stream,
                      cudaEvent_t ev_main_begin, cudaEvent_t ev_main_end, const lt_half *saved_p = nullptr) {
    // saved_p: the probability tiles of lt_attn_save_p; LSE is then not needed (fp16, whole groups only)
    const int S_pad = static_cast<int>(padded_rows(S));
    // fast addressing in the two streaming kernels when nothing is padded or strided
    auto is_contig = [&](const lt_tensor_strides &st, int H) {
        const lt_tensor_strides c = contiguous_strides(H, S, D);
        return st.batch == c.batch && st.head == c.head && st.row == c.row;
    };
    const int plain_pre = (S == S_pad && is_contig(lay.d_o, Hq) && is_contig(lay.o, Hq)) ? 1 : 0;
    const int plain_fin = (S == S_pad && is_contig(lay.dq, Hq)) ? 1 : 0;
    const long long n_rows = static_cast<long long>(B) * Hq * S_pad;  // padded row space of the workspace arrays
    uint8_t *ws = static_cast<uint8_t *>(workspace);
    unsigned int *status = reinterpret_cast<unsigned int *>(ws);
    const size_t ext_bytes = round256(static_cast<size_t>(n_rows) * 16);
    uint4 *delta_ext = reinterpret_cast<uint4 *>(ws + kStatusBytes);
    uint4 *lse_ext = reinterpret_cast<uint4 *>(ws + kStatusBytes + ext_bytes);
    float *dq_acc = reinterpret_cast<float *>(ws + kStatusBytes + 2 * ext_bytes);
    const int hpi = saved_p ? Hq / Hkv : heads_per_item(B, Hq, Hkv, S, D, causal);
    const int parts = (Hq / Hkv + hpi - 1) / hpi;
    const size_t kv_floats = static_cast<size_t>(B) * Hkv * S_pad * D;
    float *dk_acc = nullptr, *dv_acc = nullptr;
    if (parts > 1) {
        dk_acc = reinterpret_cast<float *>(ws + kStatusBytes + 2 * ext_bytes + round256(static_cast<size_t>(n_rows) * D * 4));
        dv_acc = dk_acc + kv_floats;  // kv_floats * 4 is a multiple of 256 bytes
    }

    CUtensorMap mq, mk, mv, mdo;
    int rc;
    if ((rc = make_bhsd_map(&mq, Q, B, Hq, S, D, lay.q, 128, kBf16)) != LT_OK) return rc;
    if ((rc = make_bhsd_map(&mdo, dO, B, Hq, S, D, lay.d_o, 128, kBf16)) != LT_OK) return rc;
    if ((rc = make_bhsd_map(&mk, K, B, Hkv, S, D, lay.k, 128, kBf16)) != LT_OK) return rc;
    if ((rc = make_bhsd_map(&mv, V, B, Hkv, S, D, lay.v, 128, kBf16)) != LT_OK) return rc;

    cudaError_t e = cudaMemsetAsync(status, 0, kStatusBytes, stream);
    if (e != cudaSuccess) return record_cuda_error("cudaMemsetAsync(status)", e);

    const int sms = sm_count();
    constexpr int kRowsPerBlock = 8 * (32 / (D / 8)) * kPreUnroll;
    const long long want = (n_rows + kRowsPerBlock - 1) / kRowsPerBlock;
    const int pre_blocks = static_cast<int>(want < static_cast<long long>(sms) * 16 ? want : sms * 16);
    bwd_preprocess_kernel<D, kBf16><<<pre_blocks, 256, 0, stream>>>(reinterpret_cast<const __half *>(dO),
                                                             reinterpret_cast<const __half *>(O), LSE, delta_ext,
                                                             lse_ext, dq_acc, n_rows, S, S_pad, Hq, lay.d_o, lay.o, plain_pre,
                                                             1.f / scale, status, reinterpret_cast<float4 *>(dk_acc),
                                                             parts > 1 ? static_cast<long long>(kv_floats / 2) : 0LL,
                                                             reinterpret_cast<const __half *>(V),
                                                             static_cast<long long>(B) * Hkv * S, Hkv, lay.v,
                                                             is_contig(lay.v, Hkv) ? 1 : 0);
    e = cudaGetLastError();
    if (e != cudaSuccess) return record_cuda_error("bwd_preprocess_kernel launch", e);

    BwdParams prm;
    prm.lse_ext = saved_p ? reinterpret_cast<const uint4 *>(saved_p) : lse_ext;
    prm.delta_ext = delta_ext;
    prm.dq_acc = dq_acc;
    prm.dK = reinterpret_cast<__half *>(dK);
    prm.dV = reinterpret_cast<__half *>(dV);
    prm.status = status;
    prm.B = B; prm.Hq = Hq; prm.Hkv = Hkv; prm.S = S; prm.S_pad = S_pad; prm.causal = causal ? 1 : 0;
    prm.scale = scale;
    prm.dk_st = lay.dk;
    prm.dv_st = lay.dv;
    {
        // bytes one (batch, kv head) unit keeps live: K, V, the group's Q, dO (fp16) and dQ rows (fp32)
        const int G = Hq / Hkv;
        const double unit_bytes = static_cast<double>(S_pad) * D * (2.0 * 2 + 2.0 * 2 * G + 4.0 * G);
        const int n_units = B * Hkv;
        int n_batches = static_cast<int>(unit_bytes * n_units / kL2BatchBytes) + 1;
        // CTAs flow from one batch into the next, but the last batch should still offer every SM two items
        const int max_batches = (n_units * (S_pad / kTileRows) * parts) / (2 * sms);
        if (n_batches > max_batches) n_batches = max_batches;
        if (n_batches < 1) n_batches = 1;
        prm.units_per_batch = (n_units + n_batches - 1) / n_batches;
        if (parts > 1) {
            if (prm.units_per_batch > 0xFFFF || parts > 0xFF || hpi > 0x7F) {
                set_last_error("lt_attn_bwd", "shape too large for the split-group variant");
                return LT_ERR_UNSUPPORTED;
            }
            prm.units_per_batch |= (parts << 16) | (hpi << 24);
            prm.dK = reinterpret_cast<__half *>(dk_acc);
            prm.dV = reinterpret_cast<__half *>(dv_acc);
        }
    }
    const size_t smem = sizeof(BwdSmem<D>);
    auto main_kernel = parts > 1 ? bwd_main_kernel<D, kBf16, true> : bwd_main_kernel<D, kBf16, false>;
    if constexpr (!kBf16)
        if (saved_p) main_kernel = bwd_main_kernel<D, false, false, true>;
    e = cudaFuncSetAttribute(main_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return record_cuda_error("cudaFuncSetAttribute(bwd_main)", e);
    const int n_items = B * Hkv * (S_pad / kTileRows) * parts;
    const int grid = n_items < sms ? n_items : sms;  // persistent: one CTA per SM walks the item list
    if (ev_main_begin && (e = cudaEventRecord(ev_main_begin, stream)) != cudaSuccess)
        return record_cuda_error("cudaEventRecord", e);
    // programmatic stream serialisation: the kernel may start before its predecessor has finished and
    // waits inside for it (grid_dependency_wait)
    cudaLaunchAttribute pdl;
    pdl.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    pdl.val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg_main = {};
    cfg_main.gridDim = dim3(grid);
    cfg_main.blockDim = dim3(kBwdThreads);
    cfg_main.dynamicSmemBytes = smem;
    cfg_main.stream = stream;
    cfg_main.attrs = &pdl;
    cfg_main.numAttrs = 1;
    CUtensorMap mdq = mq;  // (D = 128 never touches it)
    if constexpr (D == 64)
        if ((rc = make_f32_tile_map(&mdq, dq_acc, static_cast<uint64_t>(n_rows), 64, 128)) != LT_OK) return rc;
    e = cudaLaunchKernelEx(&cfg_main, main_kernel, mq, mk, mv, mdo, prm, mdq);
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) return record_cuda_error("bwd_main_kernel launch", e);
    if (ev_main_end && (e = cudaEventRecord(ev_main_end, stream)) != cudaSuccess)
        return record_cuda_error("cudaEventRecord", e);

    const long long n_vec8 = static_cast<long long>(B) * Hq * S * D / 8;
    const long long fwant = (n_vec8 + 255) / 256;
    const int fin_blocks = static_cast<int>(fwant < static_cast<long long>(sms) * 16 ? fwant : sms * 16);
    cudaLaunchConfig_t cfg_fin = {};
    cfg_fin.gridDim = dim3(fin_blocks);
    cfg_fin.blockDim = dim3(256);
    cfg_fin.stream = stream;
    cfg_fin.attrs = &pdl;
    cfg_fin.numAttrs = 1;
    e = cudaLaunchKernelEx(&cfg_fin, bwd_finalize_kernel<kBf16>, static_cast<const float *>(dq_acc),
                           reinterpret_cast<__half *>(dQ), n_vec8, S * (D / 8), S_pad * (D / 8), D / 8, Hq, lay.dq,
                           plain_fin);
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) return record_cuda_error("bwd_finalize_kernel launch", e);
    if (parts > 1) {
        const long long kv_vec8 = static_cast<long long>(B) * Hkv * S * D / 8;
        const long long kwant = (2 * kv_vec8 + 255) / 256;
        cfg_fin.gridDim = dim3(static_cast<int>(kwant < static_cast<long long>(sms) * 16 ? kwant : sms * 16));
        e = cudaLaunchKernelEx(&cfg_fin, bwd_finalize_kv_kernel<kBf16>, static_cast<const float *>(dk_acc),
                               static_cast<const float *>(dv_acc), reinterpret_cast<__half *>(dK),
                               reinterpret_cast<__half *>(dV), kv_vec8, S * (D / 8), S_pad * (D / 8), D / 8, Hkv, lay.dk,
                               lay.dv);
        if (e == cudaSuccess) e = cudaGetLastError();
        if (e != cudaSuccess) return record_cuda_error("bwd_finalize_kv_kernel launch", e);
    }
    return LT_OK;
}

}  // namespace lt

extern "C" {

size_t lt_attn_bwd_workspace_bytes(int B, int Hq, int Hkv, int S, int D) {
    if (lt::check_shape(B, Hq, Hkv, S, D, 1.0f) != LT_OK) return 0;
    const size_t n_rows = static_cast<size_t>(B) * Hq * static_cast<size_t>(lt::padded_rows(S));
    size_t bytes = lt::kStatusBytes + 2 * lt::round256(n_rows * 16) + lt::round256(n_rows * D * 4);
    // fp32 dK / dV sums for shapes whose groups are split over work items (either mask; sized for the
    // unmasked case, which splits no less often)
    if (lt::heads_per_item(B, Hq, Hkv, S, D, 1) < Hq / Hkv || lt::heads_per_item(B, Hq, Hkv, S, D, 0) < Hq / Hkv)
        bytes += 2 * lt::round256(static_cast<size_t>(B) * Hkv * static_cast<size_t>(lt::padded_rows(S)) * D * 4);
    return bytes;
}

int lt_attn_bwd_num_launches(int B, int Hq, int Hkv, int S, int D, int causal) {
    if (lt::check_shape(B, Hq, Hkv, S, D, 1.0f) != LT_OK) return 0;
    // preprocess, main, dQ conversion; plus the dK/dV conversion when groups are split over work items
    return lt::heads_per_item(B, Hq, Hkv, S, D, causal) < Hq / Hkv ? 4 : 3;
}

static int bwd_entry(const lt_half *Q, const lt_half *K, const lt_half *V, const lt_half *O, const lt_half *dO,
                     const float *LSE, lt_half *dQ, lt_half *dK, lt_half *dV, const lt_attn_layout *layout, int B,
                     int Hq, int Hkv, int S, int D, int causal, float scale, void *workspace, size_t workspace_bytes,
                     lt_stream_t stream, lt_event_t main_begin, lt_event_t main_end, bool bf16 = false) {
    using namespace lt;
    if (!Q || !K || !V || !O || !dO || !LSE || !dQ || !dK || !dV) return LT_ERR_INVALID_ARG;
    int rc = check_shape(B, Hq, Hkv, S, D, scale);
    if (rc != LT_OK) return rc;
    const lt_attn_layout lay = layout ? *layout : contiguous_layout(Hq, Hkv, S, D);
    if (layout && (rc = check_layout(lay, D)) != LT_OK) return rc;
    const void *ptrs[] = {Q, K, V, O, dO, dQ, dK, dV};
    for (const void *ptr : ptrs)
        if (!aligned16(ptr)) return LT_ERR_UNSUPPORTED;
    if ((reinterpret_cast<uintptr_t>(LSE) & 3u) != 0) return LT_ERR_UNSUPPORTED;  // fp32, read one at a time
    if (!workspace || !aligned256(workspace) || workspace_bytes < lt_attn_bwd_workspace_bytes(B, Hq, Hkv, S, D))
        return LT_ERR_WORKSPACE;
    if ((rc = check_device()) != LT_OK) return rc;
    if (bf16) {
        if (D == 64)
            return launch_bwd<64, true>(Q, K, V, O, dO, LSE, dQ, dK, dV, lay, B, Hq, Hkv, S, causal, scale, workspace,
                                        stream, main_begin, main_end);
        return launch_bwd<128, true>(Q, K, V, O, dO, LSE, dQ, dK, dV, lay, B, Hq, Hkv, S, causal, scale, workspace,
                                     stream, main_begin, main_end);
    }
    if (D == 64)
        return launch_bwd<64, false>(Q, K, V, O, dO, LSE, dQ, dK, dV, lay, B, Hq, Hkv, S, causal, scale, workspace,
                                     stream, main_begin, main_end);
    return launch_bwd<128, false>(Q, K, V, O, dO, LSE, dQ, dK, dV, lay, B, Hq, Hkv, S, causal, scale, workspace,
                                  stream, main_begin, main_end);
}

int lt_attn_bwd_saved_p(const lt_half *Q, const lt_half *K, const lt_half *V, const lt_half *O, const lt_half *dO,
                        const lt_half *P, lt_half *dQ, lt_half *dK, lt_half *dV, int B, int Hq, int Hkv, int S, int D,
                        int causal, float scale, void *workspace, size_t workspace_bytes, lt_stream_t stream) {
    using namespace lt;
    if (!Q || !K || !V || !O || !dO || !P || !dQ || !dK || !dV) return LT_ERR_INVALID_ARG;
    int rc = check_shape(B, Hq, Hkv, S, D, scale);
    if (rc != LT_OK) return rc;
    const void *ptrs[] = {Q, K, V, O, dO, dQ, dK, dV};
    for (const void *ptr : ptrs)
        if (!aligned16(ptr)) return LT_ERR_UNSUPPORTED;
    if (!aligned256(P)) return LT_ERR_UNSUPPORTED;
    if (!workspace || !aligned256(workspace) || workspace_bytes < lt_attn_bwd_workspace_bytes(B, Hq, Hkv, S, D))
        return LT_ERR_WORKSPACE;
    if ((rc = check_device()) != LT_OK) return rc;
    const lt_attn_layout lay = contiguous_layout(Hq, Hkv, S, D);
    if (D == 64)
        return launch_bwd<64, false>(Q, K, V, O, dO, nullptr, dQ, dK, dV, lay, B, Hq, Hkv, S, causal, scale, workspace,
                                     static_cast<cudaStream_t>(stream), nullptr, nullptr, P);
    return launch_bwd<128, false>(Q, K, V, O, dO, nullptr, dQ, dK, dV, lay, B, Hq, Hkv, S, causal, scale, workspace,
                                  static_cast<cudaStream_t>(stream), nullptr, nullptr, P);
}

int lt_attn_bwd_profiled(const lt_half *Q, const lt_half *K, const lt_half *V, const lt_half *O, const lt_half *dO,
                         const float *LSE, lt_half *dQ, lt_half *dK, lt_half *dV, int B, int Hq, int Hkv, int S,
                         int D, int causal, float scale, void *workspace, size_t workspace_bytes,
                         lt_stream_t stream, lt_event_t main_begin, lt_event_t main_end) {
    return bwd_entry(Q, K, V, O, dO, LSE, dQ, dK, dV, nullptr, B, Hq, Hkv, S, D, causal, scale, workspace,
                     workspace_bytes, stream, main_begin, main_end);
}

int lt_attn_bwd_strided(const lt_half *Q, const lt_half *K, const lt_half *V, const lt_half *O, const lt_half *dO,
                        const float *LSE, lt_half *dQ, lt_half *dK, lt_half *dV, const lt_attn_layout *layout, int B,
                        int Hq, int Hkv, int S, int D, int causal, float scale, void *workspace,
                        size_t workspace_bytes, lt_stream_t stream) {
    return bwd_entry(Q, K, V, O, dO, LSE, dQ, dK, dV, layout, B, Hq, Hkv, S, D, causal, scale, workspace,
                     workspace_bytes, stream, nullptr, nullptr);
}

int lt_attn_bwd_bf16(const lt_bf16 *Q, const lt_bf16 *K, const lt_bf16 *V, const lt_bf16 *O, const lt_bf16 *dO,
                     const float *LSE, lt_bf16 *dQ, lt_bf16 *dK, lt_bf16 *dV, const lt_attn_layout *layout, int B,
                     int Hq, int Hkv, int S, int D, int causal, float scale, void *workspace,
                     size_t workspace_bytes, lt_stream_t stream) {
    return bwd_entry(Q, K, V, O, dO, LSE, dQ, dK, dV, layout, B, Hq, Hkv, S, D, causal, scale, workspace,
                     workspace_bytes, stream, nullptr, nullptr, true);
}

int lt_attn_bwd(const lt_half *Q, const lt_half *K, const lt_half *V, const lt_half *O, const lt_half *dO,
                const float *LSE, lt_half *dQ, lt_half *dK, lt_half *dV, int B, int Hq, int Hkv, int S, int D,
                int causal, float scale, void *workspace, size_t workspace_bytes, lt_stream_t stream) {
    return lt_attn_bwd_profiled(Q, K, V, O, dO, LSE, dQ, dK, dV, B, Hq, Hkv, S, D, causal, scale, workspace,
                                workspace_bytes, stream, nullptr, nullptr);
}

}  // extern "C"

// ----------------------------------------------------------------------------- backward without a caller workspace
// Scratch for lt_attn_bwd_noalloc: lives in the library image, so every GPU that loads the
// library carries these bytes until the process exits.  In host code the array's name is
// only a handle for the runtime; the address the kernels need is fetched once per device
// with cudaGetSymbolAddress.
namespace lt {
constexpr size_t kNoAllocScratchBytes = LT_ATTN_BWD_NOALLOC_MAX_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocScratchBytes];
constexpr int kNoAllocMaxDevices = 64;
static void *g_noalloc_scratch_addr[kNoAllocMaxDevices];  // device address of the array, per device ordinal
static std::mutex g_noalloc_mutex;
}  // namespace lt

extern "C" {

int lt_attn_bwd_noalloc(const lt_half *Q, const lt_half *K, const lt_half *V, const lt_half *O, const lt_half *dO,
                        const float *LSE, lt_half *dQ, lt_half *dK, lt_half *dV, int B, int Hq, int Hkv, int S, int D,
                        int causal, float scale, lt_stream_t stream) {
    using namespace lt;
    if (!Q || !K || !V || !O || !dO || !LSE || !dQ || !dK || !dV) return LT_ERR_INVALID_ARG;
    int rc = check_shape(B, Hq, Hkv, S, D, scale);
    if (rc != LT_OK) return rc;
    const size_t need = lt_attn_bwd_workspace_bytes(B, Hq, Hkv, S, D);
    if (need == 0 || need > kNoAllocScratchBytes) {
        char msg[160];
        snprintf(msg, sizeof(msg), "this shape needs %zu bytes of scratch but the built-in scratch holds %zu; "
                 "use lt_attn_bwd with a caller workspace", need, kNoAllocScratchBytes);
        set_last_error("lt_attn_bwd_noalloc", msg);
        return LT_ERR_WORKSPACE;
    }
    if ((rc = check_device()) != LT_OK) return rc;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return record_cuda_error("cudaGetDevice", e);
    if (dev < 0 || dev >= kNoAllocMaxDevices) {
        set_last_error("lt_attn_bwd_noalloc", "device ordinal out of range");
        return LT_ERR_UNSUPPORTED;
    }
    void *scratch = nullptr;
    {
        // first call on this device: look the array's device address up (no allocation happens)
        std::lock_guard<std::mutex> lock(g_noalloc_mutex);
        if (!g_noalloc_scratch_addr[dev]) {
            void *addr = nullptr;
            e = cudaGetSymbolAddress(&addr, g_noalloc_scratch);
            if (e != cudaSuccess) return record_cuda_error("cudaGetSymbolAddress(scratch)", e);
            g_noalloc_scratch_addr[dev] = addr;
        }
        scratch = g_noalloc_scratch_addr[dev];
    }
    // lt_attn_bwd clears the status block and its preprocess kernel zeroes the dQ accumulator on
    // every call, so nothing left in the scratch by an earlier call is read
    return lt_attn_bwd(Q, K, V, O, dO, LSE, dQ, dK, dV, B, Hq, Hkv, S, D, causal, scale, scratch,
                       kNoAllocScratchBytes, stream);
}

int lt_attn_bwd_noalloc_check_status(lt_stream_t stream) {
    using namespace lt;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return record_cuda_error("cudaGetDevice", e);
    void *scratch = nullptr;
    if (dev >= 0 && dev < kNoAllocMaxDevices) {
        std::lock_guard<std::mutex> lock(g_noalloc_mutex);
        scratch = g_noalloc_scratch_addr[dev];
    }
    if (!scratch) return LT_OK;  // no lt_attn_bwd_noalloc call on this device yet: nothing to report
    return lt_attn_check_status(scratch, stream);
}

}  // extern "C"
