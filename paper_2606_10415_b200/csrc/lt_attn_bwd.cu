// Attention backward (Algorithm 1 of the paper, Section 4.1) for sm_100a.
//
// Three kernels per call:
//   bwd_preprocess_kernel : delta = rowsum(dO * O), -LSE*log2(e), zero the fp32 dQ
//                           accumulator, record max |delta| and max ||dO_row||^2
//                           (together with the V tile they bound |dS|)
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
// The main kernel is warp specialised (16 warps):
//   warp 0       TMA producer: K_j, V_j once; then a two-stage ring of {Q_i, dO_i, -LSE*log2e, delta}
//   warp 1       tensor-core issuer (one thread)
//   warp 2       owns the tensor-memory allocation
//   warps 4-11   softmax / dS warps: warps 4-7 take query columns 0-63 of a tile pair,
//                warps 8-11 columns 64-127; each thread owns one key row
//   warps 12-15  dQ reduction: tensor memory -> fp32 red.global into the accumulator
// Transposed scores are used (S^T = K Q^T, dP^T = V dO^T) so that P^T, written back to
// tensor memory as fp16, is directly the A operand of dV += P^T dO; dS^T goes through
// shared memory once and serves both dK += dS^T Q (contraction-contiguous A) and
// dQ = dS K (row-contracted A).
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
    kWaitDkvFull = 211, kBadSmemAlign = 220
};

// ----------------------------------------------------------------------------- preprocess
// One half-warp (D = 128) or quarter-warp (D = 64) per row: 16-byte loads of dO and O.
template <int D>
__global__ void __launch_bounds__(256)
bwd_preprocess_kernel(const __half *__restrict__ dO, const __half *__restrict__ O, const float *__restrict__ lse,
                      float *__restrict__ delta, float *__restrict__ neg_lse_log2, float *__restrict__ dq_acc,
                      long long n_rows, unsigned int *status) {
    constexpr int kLanesPerRow = D / 8;
    constexpr int kRowsPerWarp = 32 / kLanesPerRow;
    const int lane = threadIdx.x & 31;
    const int sub = lane % kLanesPerRow;
    const long long warp_global = (static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5;
    const long long n_warps = (static_cast<long long>(gridDim.x) * blockDim.x) >> 5;
    float max_abs_delta = 0.f, max_norm2 = 0.f;
    for (long long row0 = warp_global * kRowsPerWarp; row0 < n_rows; row0 += n_warps * kRowsPerWarp) {
        const long long row = row0 + lane / kLanesPerRow;
        float acc = 0.f, n2 = 0.f;
        if (row < n_rows) {
            const uint4 a = __ldg(reinterpret_cast<const uint4 *>(dO + row * D) + sub);
            const uint4 b = __ldg(reinterpret_cast<const uint4 *>(O + row * D) + sub);
            const __half2 *ah = reinterpret_cast<const __half2 *>(&a);
            const __half2 *bh = reinterpret_cast<const __half2 *>(&b);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float2 x = __half22float2(ah[e]);
                const float2 y = __half22float2(bh[e]);
                acc = fmaf(x.x, y.x, acc);
                acc = fmaf(x.y, y.y, acc);
                n2 = fmaf(x.x, x.x, n2);
                n2 = fmaf(x.y, x.y, n2);
            }
            float4 *z = reinterpret_cast<float4 *>(dq_acc + row * D) + sub * 2;
            z[0] = make_float4(0.f, 0.f, 0.f, 0.f);
            z[1] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int off = kLanesPerRow / 2; off > 0; off >>= 1) {
            acc += __shfl_xor_sync(0xffffffffu, acc, off);
            n2 += __shfl_xor_sync(0xffffffffu, n2, off);
        }
        if (row < n_rows) {
            if (sub == 0) {
                delta[row] = acc;
                neg_lse_log2[row] = -lse[row] * kLog2e;
            }
            max_abs_delta = fmaxf(max_abs_delta, fabsf(acc));
            max_norm2 = fmaxf(max_norm2, n2);
        }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        max_abs_delta = fmaxf(max_abs_delta, __shfl_xor_sync(0xffffffffu, max_abs_delta, off));
        max_norm2 = fmaxf(max_norm2, __shfl_xor_sync(0xffffffffu, max_norm2, off));
    }
    if (lane == 0) {
        // non-negative floats order like their bit patterns; NaN/inf inputs simply saturate the bound
        atomicMax(status + kStatusWordMaxAbsDelta, __float_as_uint(max_abs_delta));
        atomicMax(status + kStatusWordMaxDoNorm2, __float_as_uint(max_norm2));
    }
}

// ----------------------------------------------------------------------------- finalize
__global__ void __launch_bounds__(256)
bwd_finalize_kernel(const float *__restrict__ dq_acc, __half *__restrict__ dQ, long long n_vec8) {
    const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
    for (long long v = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; v < n_vec8; v += stride) {
        const float4 a = __ldcs(reinterpret_cast<const float4 *>(dq_acc) + 2 * v);
        const float4 b = __ldcs(reinterpret_cast<const float4 *>(dq_acc) + 2 * v + 1);
        uint4 o;
        o.x = pack_half2(a.x, a.y);
        o.y = pack_half2(a.z, a.w);
        o.z = pack_half2(b.x, b.y);
        o.w = pack_half2(b.z, b.w);
        reinterpret_cast<uint4 *>(dQ)[v] = o;
    }
}

// ----------------------------------------------------------------------------- main kernel
constexpr int kStages = 2;
constexpr int kBwdThreads = 512;
constexpr int kComputeWarp0 = 4, kNumComputeWarps = 8;
constexpr int kReduceWarp0 = 12, kNumReduceWarps = 4;

template <int D>
struct BwdSmem {
    static constexpr int kBoxes = D / 64;
    static constexpr int kTile = kBoxes * kBoxBytesBwd;
    uint8_t k[kTile];
    uint8_t v[kTile];
    uint8_t q[kStages][kTile];
    uint8_t d_o[kStages][kTile];
    uint8_t ds[2 * kBoxBytesBwd];           // dS^T: rows = key index, 128 query columns in two swizzled tiles
    float neg_lse_log2[kStages][kTileRows]; // -LSE * log2(e) of the stage's query tile
    float delta[kStages][kTileRows];
    uint64_t bar_kv;
    uint64_t bar_stage_full[kStages], bar_stage_empty[kStages];
    uint64_t bar_s_full, bar_p_ready, bar_dp_full, bar_ds_ready, bar_ds_free, bar_dq_full, bar_dq_empty, bar_dkv_full;
    float red[4];
    float ds_mult;
    uint32_t tmem_base;
    int abort_flag;
};

struct BwdParams {
    const float *neg_lse_log2;
    const float *delta;
    float *dq_acc;
    __half *dK;
    __half *dV;
    unsigned int *status;
    int B, Hq, Hkv, S, causal;
    float scale;
};

template <int D>
__global__ void __launch_bounds__(kBwdThreads, 1)
bwd_main_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_do,
                const BwdParams p) {
    using Smem = BwdSmem<D>;
    constexpr int kBoxes = D / 64;
    constexpr uint32_t kTileBytes = kBoxes * kBoxBytesBwd;
    constexpr uint32_t kStageBytes = 2 * kTileBytes + 2 * kTileRows * sizeof(float);
    constexpr uint32_t kTmemCols = 512;
    constexpr uint32_t kColS = 0, kColdP = 128, kColdV = 256, kColdK = 384;

    extern __shared__ __align__(1024) uint8_t smem_raw[];
    Smem &sm = *reinterpret_cast<Smem *>(smem_raw);
    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;

    // work item: key tile j of (batch b, kv head g); heavy (small j) items get the low block ids
    const int n_tiles = p.S / kTileRows;
    const int G = p.Hq / p.Hkv;
    const int n_bg = p.B * p.Hkv;
    const int j = blockIdx.x / n_bg;
    const int bg = blockIdx.x % n_bg;
    const int b = bg / p.Hkv;
    const int g = bg % p.Hkv;
    const int i_first = p.causal ? j : 0;
    const int tiles_per_head = n_tiles - i_first;
    const int n_iter = G * tiles_per_head;  // flattened (query head of the group, query tile) loop
    const int kv_row0 = (b * p.Hkv + g) * p.S + j * kTileRows;

    // the swizzled tiles need 1024-byte alignment; the shared window is expected to give it
    const bool smem_ok = (smem_u32(smem_raw) & 1023u) == 0u;
    if (tid == 0) {
        sm.abort_flag = smem_ok ? 0 : 1;
        if (!smem_ok) atomicCAS(p.status + kStatusWordTimeout, 0u, static_cast<unsigned int>(kBadSmemAlign));
        mbar_init(&sm.bar_kv, 1);
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&sm.bar_stage_full[s], 1);
            mbar_init(&sm.bar_stage_empty[s], 1);
        }
        mbar_init(&sm.bar_s_full, 1);
        mbar_init(&sm.bar_p_ready, kNumComputeWarps);
        mbar_init(&sm.bar_dp_full, 1);
        mbar_init(&sm.bar_ds_ready, kNumComputeWarps);
        mbar_init(&sm.bar_ds_free, 1);
        mbar_init(&sm.bar_dq_full, 1);
        mbar_init(&sm.bar_dq_empty, kNumReduceWarps);
        mbar_init(&sm.bar_dkv_full, 1);
        mbar_fence_init();
        tma_prefetch_desc(&map_q);
        tma_prefetch_desc(&map_k);
        tma_prefetch_desc(&map_v);
        tma_prefetch_desc(&map_do);
    }
    if (warp == 2) {
        tmem_alloc(&sm.tmem_base, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = sm.tmem_base;
    volatile int *abort_flag = &sm.abort_flag;

    // iteration n -> first row of its query tile in the [B*Hq*S, D] view
    auto q_row_of = [&](int n) -> long long {
        const int hh = n / tiles_per_head;
        const int i = i_first + (n - hh * tiles_per_head);
        return (static_cast<long long>(b) * p.Hq + g * G + hh) * p.S + static_cast<long long>(i) * kTileRows;
    };

    // ---- K_j and V_j are requested before anything else
    if (warp == 0 && lane == 0 && smem_ok) {
        mbar_arrive_expect_tx(&sm.bar_kv, 2 * kTileBytes);
#pragma unroll
        for (int x = 0; x < kBoxes; ++x) {
            tma_load_2d(sm.k + x * kBoxBytesBwd, &map_k, &sm.bar_kv, x * 64, kv_row0);
            tma_load_2d(sm.v + x * kBoxBytesBwd, &map_v, &sm.bar_kv, x * 64, kv_row0);
        }
    }

    // Power-of-two factor applied to dS before it is rounded to fp16, chosen from a bound
    // on |dS| <= |dP| + |delta| <= max||dO_row|| * max||V_row|| + max|delta| so that the scaled
    // values use fp16's normal range without overflow.  Undone exactly in the dQ/dK epilogues.
    if (warp >= kComputeWarp0 && warp < kComputeWarp0 + 4) {
        const int row = tid - kComputeWarp0 * 32;
        float n2 = 0.f;
        if (mbar_wait(&sm.bar_kv, 0, abort_flag, p.status, kWaitKV)) {
#pragma unroll
            for (int x = 0; x < kBoxes; ++x) {
                const uint4 *src = reinterpret_cast<const uint4 *>(sm.v + x * kBoxBytesBwd + row * 128);
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    const uint4 u = src[c];
                    const __half2 *h = reinterpret_cast<const __half2 *>(&u);
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float2 f = __half22float2(h[e]);
                        n2 = fmaf(f.x, f.x, n2);
                        n2 = fmaf(f.y, f.y, n2);
                    }
                }
            }
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) n2 = fmaxf(n2, __shfl_xor_sync(0xffffffffu, n2, off));
        if (lane == 0) sm.red[warp - kComputeWarp0] = n2;
    }
    __syncthreads();
    if (tid == 0) {
        const float vmax2 = fmaxf(fmaxf(sm.red[0], sm.red[1]), fmaxf(sm.red[2], sm.red[3]));
        const float do2 = __uint_as_float(p.status[kStatusWordMaxDoNorm2]);
        const float dmax = __uint_as_float(p.status[kStatusWordMaxAbsDelta]);
        const float bound = sqrtf(do2) * sqrtf(vmax2) + dmax;
        int e = 24;                                  // all-zero dO: any factor works
        if (!(bound < 3.0e38f)) e = -14;             // inf/NaN inputs: outputs are non-finite anyway
        else if (bound > 1e-30f) e = min(24, max(-14, ilogbf(32768.f / bound)));
        sm.ds_mult = ldexpf(1.f, e);
    }
    __syncthreads();
    const float ds_mult = sm.ds_mult;
    const float dq_mult = p.scale / ds_mult;

    if (warp == 0) {
        // ================================================================= TMA producer
        if (lane == 0 && smem_ok) {
            int issued = 0;
            for (int n = 0; n < n_iter; ++n) {
                const int s = n & 1, k = n >> 1;
                if (k >= 1 && !mbar_wait(&sm.bar_stage_empty[s], (k - 1) & 1, abort_flag, p.status, kWaitStageEmpty))
                    break;
                const long long q_row0 = q_row_of(n);
                mbar_arrive_expect_tx(&sm.bar_stage_full[s], kStageBytes);
#pragma unroll
                for (int x = 0; x < kBoxes; ++x) {
                    tma_load_2d(sm.q[s] + x * kBoxBytesBwd, &map_q, &sm.bar_stage_full[s], x * 64,
                                static_cast<int>(q_row0));
                    tma_load_2d(sm.d_o[s] + x * kBoxBytesBwd, &map_do, &sm.bar_stage_full[s], x * 64,
                                static_cast<int>(q_row0));
                }
                bulk_load_1d(sm.neg_lse_log2[s], p.neg_lse_log2 + q_row0, kTileRows * sizeof(float),
                             &sm.bar_stage_full[s]);
                bulk_load_1d(sm.delta[s], p.delta + q_row0, kTileRows * sizeof(float), &sm.bar_stage_full[s]);
                issued = n + 1;
            }
            if (*abort_flag) {
                // abandoned: give this CTA's own copies a bounded time to land before shared memory is released
                for (int t = 0; t < (1 << 16) && !mbar_try_wait(&sm.bar_kv, 0); ++t) {}
                for (int n = max(0, issued - kStages); n < issued; ++n)
                    for (int t = 0; t < (1 << 16) && !mbar_try_wait(&sm.bar_stage_full[n & 1], (n >> 1) & 1); ++t) {}
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ================================================================= tensor-core issuer
        if (lane == 0 && smem_ok) {
            const uint32_t sK = smem_u32(sm.k), sV = smem_u32(sm.v), sdS = smem_u32(sm.ds);
            constexpr uint32_t idesc_s = make_idesc(128, 128, false, false);
            constexpr uint32_t idesc_dv = make_idesc(128, D, false, true);
            constexpr uint32_t idesc_dq = make_idesc(128, D, true, true);
            auto issue_s = [&](int n) {  // S^T = K_j Q_i^T
                const uint32_t sQn = smem_u32(sm.q[n & 1]);
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint32_t koff = (kk >> 2) * kBoxBytesBwd + (kk & 3) * 32;
                    umma_ss(tmem + kColS, desc_kmajor(sK + koff), desc_kmajor(sQn + koff), idesc_s, kk > 0);
                }
                umma_commit(&sm.bar_s_full);
            };
            bool ok = mbar_wait(&sm.bar_kv, 0, abort_flag, p.status, kWaitKV) &&
                      mbar_wait(&sm.bar_stage_full[0], 0, abort_flag, p.status, kWaitStageFull);
            if (ok) {
                tc_fence_after_sync();
                issue_s(0);
            }
            for (int n = 0; n < n_iter && ok; ++n) {
                const int s = n & 1;
                const uint32_t sQ = smem_u32(sm.q[s]), sdO = smem_u32(sm.d_o[s]);
                // dP^T = V_j dO_i^T   (its columns held the previous dQ partial until the reduce warps drained it)
                if (n > 0 && !(ok = mbar_wait(&sm.bar_dq_empty, (n - 1) & 1, abort_flag, p.status, kWaitDqEmpty))) break;
                tc_fence_after_sync();
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint32_t koff = (kk >> 2) * kBoxBytesBwd + (kk & 3) * 32;
                    umma_ss(tmem + kColdP, desc_kmajor(sV + koff), desc_kmajor(sdO + koff), idesc_s, kk > 0);
                }
                umma_commit(&sm.bar_dp_full);
                // dV_j += P^T dO_i   (A = P^T from tensor memory; query columns 0-63 sit at columns 0-31,
                //                     query columns 64-127 at columns 64-95 of the S region)
                if (!(ok = mbar_wait(&sm.bar_p_ready, n & 1, abort_flag, p.status, kWaitPReady))) break;
                tc_fence_after_sync();
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)
                    umma_ts(tmem + kColdV, tmem + kColS + (kk >> 2) * 64 + (kk & 3) * 8,
                            desc_mnmajor(sdO + kk * 2048, kBoxBytesBwd), idesc_dv, (n > 0) | (kk > 0));
                // the next S^T overwrites P^T; the tensor pipe executes in issue order
                if (n + 1 < n_iter) {
                    if (!(ok = mbar_wait(&sm.bar_stage_full[(n + 1) & 1], ((n + 1) >> 1) & 1, abort_flag, p.status,
                                         kWaitStageFull)))
                        break;
                    issue_s(n + 1);
                }
                if (!(ok = mbar_wait(&sm.bar_ds_ready, n & 1, abort_flag, p.status, kWaitDsReady))) break;
                tc_fence_after_sync();
                // dQ_i partial = dS K_j   (contraction over key rows; lands on the dP columns)
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)
                    umma_ss(tmem + kColdP, desc_mnmajor(sdS + kk * 2048, kBoxBytesBwd),
                            desc_mnmajor(sK + kk * 2048, kBoxBytesBwd), idesc_dq, kk > 0);
                umma_commit(&sm.bar_dq_full);
                // dK_j += dS^T Q_i
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {
                    const uint32_t koff = (kk >> 2) * kBoxBytesBwd + (kk & 3) * 32;
                    umma_ss(tmem + kColdK, desc_kmajor(sdS + koff), desc_mnmajor(sQ + kk * 2048, kBoxBytesBwd),
                            idesc_dv, (n > 0) | (kk > 0));
                }
                umma_commit(&sm.bar_stage_empty[s]);
                umma_commit(&sm.bar_ds_free);
            }
            if (ok) umma_commit(&sm.bar_dkv_full);
        }
        __syncwarp();
    } else if (warp >= kComputeWarp0 && warp < kComputeWarp0 + kNumComputeWarps) {
        // ================================================================= softmax / dS warps
        const int quad = warp & 3;                           // tensor-memory lane quadrant
        const int half_sel = (warp - kComputeWarp0) >> 2;    // 0: query columns 0-63, 1: 64-127
        const int row = quad * 32 + lane;                    // key row inside the tile
        const uint32_t lane_base = static_cast<uint32_t>(quad * 32) << 16;
        const uint32_t cbase = half_sel * 64;
        const float scale_log2 = p.scale * kLog2e;
        uint8_t *ds_tile = sm.ds + half_sel * kBoxBytesBwd;
        uint32_t pp[32];  // this thread's 64 P^T values of the current tile pair, packed fp16 pairs
        bool ok = smem_ok;

        auto compute_p = [&](int n) -> bool {
            const int s = n & 1;
            if (!mbar_wait(&sm.bar_stage_full[s], (n >> 1) & 1, abort_flag, p.status, kWaitStageFull)) return false;
            if (!mbar_wait(&sm.bar_s_full, n & 1, abort_flag, p.status, kWaitSFull)) return false;
            tc_fence_after_sync();
            const int hh = n / tiles_per_head;
            const bool diag = p.causal && (i_first + (n - hh * tiles_per_head) == j);
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                uint32_t sv[32];
                tmem_ld32(tmem + lane_base + kColS + cbase + c * 32, sv);
                tmem_wait_ld();
#pragma unroll
                for (int e = 0; e < 32; e += 4) {
                    const int q0 = cbase + c * 32 + e;
                    const float4 nl = *reinterpret_cast<const float4 *>(&sm.neg_lse_log2[s][q0]);
                    float p0 = fast_exp2(fmaf(__uint_as_float(sv[e]), scale_log2, nl.x));
                    float p1 = fast_exp2(fmaf(__uint_as_float(sv[e + 1]), scale_log2, nl.y));
                    float p2 = fast_exp2(fmaf(__uint_as_float(sv[e + 2]), scale_log2, nl.z));
                    float p3 = fast_exp2(fmaf(__uint_as_float(sv[e + 3]), scale_log2, nl.w));
                    if (diag) {  // key row is hidden from query column q when row > q
                        if (row > q0) p0 = 0.f;
                        if (row > q0 + 1) p1 = 0.f;
                        if (row > q0 + 2) p2 = 0.f;
                        if (row > q0 + 3) p3 = 0.f;
                    }
                    pp[c * 16 + e / 2] = pack_half2(p0, p1);
                    pp[c * 16 + e / 2 + 1] = pack_half2(p2, p3);
                }
                uint32_t out[16];
#pragma unroll
                for (int e = 0; e < 16; ++e) out[e] = pp[c * 16 + e];
                // in place: these 16 columns were read by this thread in this or the previous chunk
                tmem_st16(tmem + lane_base + kColS + cbase + c * 16, out);
            }
            tmem_wait_st();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.bar_p_ready);
            return true;
        };

        ok = ok && compute_p(0);
        for (int n = 0; n < n_iter && ok; ++n) {
            const int s = n & 1;
            if (!(ok = mbar_wait(&sm.bar_dp_full, n & 1, abort_flag, p.status, kWaitDpFull))) break;
            tc_fence_after_sync();
            uint32_t o[32];
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                uint32_t dp[32];
                tmem_ld32(tmem + lane_base + kColdP + cbase + c * 32, dp);
                tmem_wait_ld();
#pragma unroll
                for (int e = 0; e < 32; e += 4) {
                    const int q0 = cbase + c * 32 + e;
                    const float4 dl = *reinterpret_cast<const float4 *>(&sm.delta[s][q0]);
                    const float2 pa = __half22float2(*reinterpret_cast<const __half2 *>(&pp[c * 16 + e / 2]));
                    const float2 pb = __half22float2(*reinterpret_cast<const __half2 *>(&pp[c * 16 + e / 2 + 1]));
                    const float d0 = pa.x * ds_mult * (__uint_as_float(dp[e]) - dl.x);
                    const float d1 = pa.y * ds_mult * (__uint_as_float(dp[e + 1]) - dl.y);
                    const float d2 = pb.x * ds_mult * (__uint_as_float(dp[e + 2]) - dl.z);
                    const float d3 = pb.y * ds_mult * (__uint_as_float(dp[e + 3]) - dl.w);
                    o[c * 16 + e / 2] = pack_half2(d0, d1);
                    o[c * 16 + e / 2 + 1] = pack_half2(d2, d3);
                }
            }
            // the previous dS^T tile must have been consumed by dQ and dK before it is overwritten
            if (n > 0 && !(ok = mbar_wait(&sm.bar_ds_free, (n - 1) & 1, abort_flag, p.status, kWaitDsFree))) break;
            // 64 query columns = eight 16-byte chunks of row `row` in this half's tile
#pragma unroll
            for (int v4 = 0; v4 < 8; ++v4)
                *reinterpret_cast<uint4 *>(ds_tile + swz128_offset(row, v4 * 8)) =
                    make_uint4(o[4 * v4], o[4 * v4 + 1], o[4 * v4 + 2], o[4 * v4 + 3]);
            fence_proxy_async_smem();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.bar_ds_ready);
            if (n + 1 < n_iter) ok = compute_p(n + 1);
        }

        // epilogue: warps 4-7 write dK_j, warps 8-11 write dV_j; thread = key row
        if (ok && mbar_wait(&sm.bar_dkv_full, 0, abort_flag, p.status, kWaitDkvFull)) {
            tc_fence_after_sync();
            const float mult = half_sel == 0 ? dq_mult : 1.f;
            const uint32_t col0 = half_sel == 0 ? kColdK : kColdV;
            __half *dst = (half_sel == 0 ? p.dK : p.dV) + (static_cast<long long>(kv_row0) + row) * D;
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
                uint32_t r[32];
                tmem_ld32(tmem + lane_base + col0 + c * 32, r);
                tmem_wait_ld();
#pragma unroll
                for (int v8 = 0; v8 < 4; ++v8) {
                    uint4 w;
                    w.x = pack_half2(__uint_as_float(r[8 * v8 + 0]) * mult, __uint_as_float(r[8 * v8 + 1]) * mult);
                    w.y = pack_half2(__uint_as_float(r[8 * v8 + 2]) * mult, __uint_as_float(r[8 * v8 + 3]) * mult);
                    w.z = pack_half2(__uint_as_float(r[8 * v8 + 4]) * mult, __uint_as_float(r[8 * v8 + 5]) * mult);
                    w.w = pack_half2(__uint_as_float(r[8 * v8 + 6]) * mult, __uint_as_float(r[8 * v8 + 7]) * mult);
                    reinterpret_cast<uint4 *>(dst + c * 32)[v8] = w;
                }
            }
        }
    } else if (warp >= kReduceWarp0) {
        // ================================================================= dQ reduction warps
        const int quad = warp & 3;
        bool ok = smem_ok;
        for (int n = 0; n < n_iter && ok; ++n) {
            if (!(ok = mbar_wait(&sm.bar_dq_full, n & 1, abort_flag, p.status, kWaitDqFull))) break;
            tc_fence_after_sync();
            float *dq_tile = p.dq_acc + q_row_of(n) * D;
#pragma unroll
            for (int ch = 0; ch < D / 64; ++ch) {
                uint32_t r[2][32];
#pragma unroll
                for (int lh = 0; lh < 2; ++lh)
                    tmem_ld_16x256b_x8(tmem + (static_cast<uint32_t>(quad * 32 + lh * 16) << 16) + kColdP + ch * 64,
                                       r[lh]);
                tmem_wait_ld();
                if (ch == D / 64 - 1) {
                    // the whole partial is in registers: the dP columns may be overwritten
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&sm.bar_dq_empty);
                }
                // four neighbouring threads add 32 contiguous bytes of one query row
#pragma unroll
                for (int lh = 0; lh < 2; ++lh) {
                    float *base = dq_tile + static_cast<long long>(quad * 32 + lh * 16 + (lane >> 2)) * D + ch * 64 +
                                  2 * (lane & 3);
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        red_add_v2(base + 8 * k, __uint_as_float(r[lh][4 * k]) * dq_mult,
                                   __uint_as_float(r[lh][4 * k + 1]) * dq_mult);
                        red_add_v2(base + 8 * D + 8 * k, __uint_as_float(r[lh][4 * k + 2]) * dq_mult,
                                   __uint_as_float(r[lh][4 * k + 3]) * dq_mult);
                    }
                }
            }
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == 2) tmem_dealloc(tmem, kTmemCols);
}

template <int D>
static int launch_bwd(const lt_half *Q, const lt_half *K, const lt_half *V, const lt_half *O, const lt_half *dO,
                      const float *LSE, lt_half *dQ, lt_half *dK, lt_half *dV, int B, int Hq, int Hkv, int S,
                      int causal, float scale, void *workspace, cudaStream_t stream, cudaEvent_t ev_main_begin,
                      cudaEvent_t ev_main_end) {
    const long long n_rows = static_cast<long long>(B) * Hq * S;
    uint8_t *ws = static_cast<uint8_t *>(workspace);
    unsigned int *status = reinterpret_cast<unsigned int *>(ws);
    const size_t row_bytes = round256(static_cast<size_t>(n_rows) * 4);
    float *delta = reinterpret_cast<float *>(ws + kStatusBytes);
    float *neg_lse_log2 = reinterpret_cast<float *>(ws + kStatusBytes + row_bytes);
    float *dq_acc = reinterpret_cast<float *>(ws + kStatusBytes + 2 * row_bytes);

    CUtensorMap mq, mk, mv, mdo;
    int rc;
    if ((rc = make_tile_map(&mq, Q, n_rows, D, 128)) != LT_OK) return rc;
    if ((rc = make_tile_map(&mdo, dO, n_rows, D, 128)) != LT_OK) return rc;
    if ((rc = make_tile_map(&mk, K, static_cast<uint64_t>(B) * Hkv * S, D, 128)) != LT_OK) return rc;
    if ((rc = make_tile_map(&mv, V, static_cast<uint64_t>(B) * Hkv * S, D, 128)) != LT_OK) return rc;

    cudaError_t e = cudaMemsetAsync(status, 0, kStatusBytes, stream);
    if (e != cudaSuccess) return record_cuda_error("cudaMemsetAsync(status)", e);

    int sms = 148;
    {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    }
    constexpr int kRowsPerBlock = 8 * (32 / (D / 8));
    const long long want = (n_rows + kRowsPerBlock - 1) / kRowsPerBlock;
    const int pre_blocks = static_cast<int>(want < static_cast<long long>(sms) * 16 ? want : sms * 16);
    bwd_preprocess_kernel<D><<<pre_blocks, 256, 0, stream>>>(reinterpret_cast<const __half *>(dO),
                                                             reinterpret_cast<const __half *>(O), LSE, delta,
                                                             neg_lse_log2, dq_acc, n_rows, status);
    e = cudaGetLastError();
    if (e != cudaSuccess) return record_cuda_error("bwd_preprocess_kernel launch", e);

    BwdParams prm;
    prm.neg_lse_log2 = neg_lse_log2;
    prm.delta = delta;
    prm.dq_acc = dq_acc;
    prm.dK = reinterpret_cast<__half *>(dK);
    prm.dV = reinterpret_cast<__half *>(dV);
    prm.status = status;
    prm.B = B; prm.Hq = Hq; prm.Hkv = Hkv; prm.S = S; prm.causal = causal ? 1 : 0;
    prm.scale = scale;
    const size_t smem = sizeof(BwdSmem<D>);
    e = cudaFuncSetAttribute(bwd_main_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return record_cuda_error("cudaFuncSetAttribute(bwd_main)", e);
    const int grid = B * Hkv * (S / kTileRows);
    if (ev_main_begin && (e = cudaEventRecord(ev_main_begin, stream)) != cudaSuccess)
        return record_cuda_error("cudaEventRecord", e);
    bwd_main_kernel<D><<<grid, kBwdThreads, smem, stream>>>(mq, mk, mv, mdo, prm);
    e = cudaGetLastError();
    if (e != cudaSuccess) return record_cuda_error("bwd_main_kernel launch", e);
    if (ev_main_end && (e = cudaEventRecord(ev_main_end, stream)) != cudaSuccess)
        return record_cuda_error("cudaEventRecord", e);

    const long long n_vec8 = n_rows * D / 8;
    const long long fwant = (n_vec8 + 255) / 256;
    const int fin_blocks = static_cast<int>(fwant < static_cast<long long>(sms) * 16 ? fwant : sms * 16);
    bwd_finalize_kernel<<<fin_blocks, 256, 0, stream>>>(dq_acc, reinterpret_cast<__half *>(dQ), n_vec8);
    e = cudaGetLastError();
    if (e != cudaSuccess) return record_cuda_error("bwd_finalize_kernel launch", e);
    return LT_OK;
}

}  // namespace lt

extern "C" {

size_t lt_attn_bwd_workspace_bytes(int B, int Hq, int Hkv, int S, int D) {
    if (lt::check_shape(B, Hq, Hkv, S, D, 1.0f) != LT_OK) return 0;
    const size_t n_rows = static_cast<size_t>(B) * Hq * S;
    return lt::kStatusBytes + 2 * lt::round256(n_rows * 4) + lt::round256(n_rows * D * 4);
}

int lt_attn_bwd_num_launches(void) { return 3; }

int lt_attn_bwd_profiled(const lt_half *Q, const lt_half *K, const lt_half *V, const lt_half *O, const lt_half *dO,
                         const float *LSE, lt_half *dQ, lt_half *dK, lt_half *dV, int B, int Hq, int Hkv, int S,
                         int D, int causal, float scale, void *workspace, size_t workspace_bytes,
                         lt_stream_t stream, lt_event_t main_begin, lt_event_t main_end) {
    using namespace lt;
    if (!Q || !K || !V || !O || !dO || !LSE || !dQ || !dK || !dV) return LT_ERR_INVALID_ARG;
    int rc = check_shape(B, Hq, Hkv, S, D, scale);
    if (rc != LT_OK) return rc;
    const void *ptrs[] = {Q, K, V, O, dO, LSE, dQ, dK, dV};
    for (const void *ptr : ptrs)
        if (!aligned16(ptr)) return LT_ERR_UNSUPPORTED;
    if (!workspace || !aligned256(workspace) || workspace_bytes < lt_attn_bwd_workspace_bytes(B, Hq, Hkv, S, D))
        return LT_ERR_WORKSPACE;
    if ((rc = check_device()) != LT_OK) return rc;
    if (D == 64)
        return launch_bwd<64>(Q, K, V, O, dO, LSE, dQ, dK, dV, B, Hq, Hkv, S, causal, scale, workspace, stream,
                              main_begin, main_end);
    return launch_bwd<128>(Q, K, V, O, dO, LSE, dQ, dK, dV, B, Hq, Hkv, S, causal, scale, workspace, stream,
                           main_begin, main_end);
}

int lt_attn_bwd(const lt_half *Q, const lt_half *K, const lt_half *V, const lt_half *O, const lt_half *dO,
                const float *LSE, lt_half *dQ, lt_half *dK, lt_half *dV, int B, int Hq, int Hkv, int S, int D,
                int causal, float scale, void *workspace, size_t workspace_bytes, lt_stream_t stream) {
    return lt_attn_bwd_profiled(Q, K, V, O, dO, LSE, dQ, dK, dV, B, Hq, Hkv, S, D, causal, scale, workspace,
                                workspace_bytes, stream, nullptr, nullptr);
}

}  // extern "C"
