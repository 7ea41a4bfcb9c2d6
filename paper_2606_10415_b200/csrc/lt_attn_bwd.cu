// Attention backward (Algorithm 1 of the paper, Section 4.1) for sm_100a.
//
// Three kernels per call:
//   bwd_preprocess_kernel : delta = rowsum(dO * O), zero the fp32 dQ accumulator,
//                           record max |delta| and max ||dO_row||^2 (they bound dS)
//   bwd_main_kernel       : per (batch, kv head, key tile j): loop over the group's
//                           query heads and the visible query tiles i, recompute
//                           P^T from LSE, and run the five tile contractions on
//                           tcgen05 tensor cores with tensor-memory accumulators
//   bwd_finalize_kernel   : dQ fp32 accumulator -> fp16
//
// Loop order differs from Algorithm 1 (which is query-outer and reduces dK/dV partials
// across workers): here a CTA owns one key/value tile, keeps dK_j and dV_j resident in
// tensor memory for the whole loop, and the cross-CTA reduction falls on dQ instead.
#include "lt_common.cuh"
#include "lt_host.h"

namespace lt {

constexpr int kTileRows = 128;             // rows of a query tile and of a key/value tile
constexpr int kBoxBytesBwd = 128 * 128;    // one swizzled tile of 128 rows x 64 fp16
constexpr float kLog2e = 1.4426950408889634f;

// wait codes recorded in the status block when a bounded wait gives up
enum { kWaitKV = 201, kWaitQdO = 202, kWaitMma1 = 203, kWaitMma2 = 204 };

// ----------------------------------------------------------------------------- preprocess
// One half-warp (D = 128) or quarter-warp (D = 64) per row: 16-byte loads of dO and O.
template <int D>
__global__ void __launch_bounds__(256)
bwd_preprocess_kernel(const __half *__restrict__ dO, const __half *__restrict__ O, float *__restrict__ delta,
                      float *__restrict__ dq_acc, long long n_rows, unsigned int *status) {
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
            if (sub == 0) delta[row] = acc;
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
template <int D>
struct __align__(1024) BwdSmem {
    static constexpr int kBoxes = D / 64;
    uint8_t k[kBoxes * kBoxBytesBwd];
    uint8_t v[kBoxes * kBoxBytesBwd];
    uint8_t q[kBoxes * kBoxBytesBwd];
    uint8_t d_o[kBoxes * kBoxBytesBwd];
    uint8_t ds[2 * kBoxBytesBwd];   // dS^T: rows = key index, 128 query columns in two swizzled tiles
    float neg_lse_log2[kTileRows];  // -LSE * log2(e) of the current query tile
    float delta[kTileRows];
    float red[4];
    uint64_t bar_kv, bar_qdo, bar_mma;
    uint32_t tmem_base;
    int abort_flag;
};

__device__ __forceinline__ void red_add_v4(float *addr, float a, float b, float c, float d) {
    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(addr), "f"(a), "f"(b), "f"(c), "f"(d)
                 : "memory");
}

struct BwdParams {
    const float *lse;
    const float *delta;
    float *dq_acc;
    __half *dK;
    __half *dV;
    unsigned int *status;
    int B, Hq, Hkv, S, causal;
    float scale;
};

template <int D>
__global__ void __launch_bounds__(128, 1)
bwd_main_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_do,
                const BwdParams p) {
    using Smem = BwdSmem<D>;
    constexpr int kBoxes = D / 64;
    constexpr uint32_t kTileBytes = kBoxes * kBoxBytesBwd;
    constexpr uint32_t kTmemCols = 512;
    constexpr uint32_t kColS = 0, kColdP = 128, kColdV = 256, kColdK = 384;

    extern __shared__ uint8_t smem_raw[];
    Smem &sm = *reinterpret_cast<Smem *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
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

    if (tid == 0) {
        sm.abort_flag = 0;
        mbar_init(&sm.bar_kv, 1);
        mbar_init(&sm.bar_qdo, 1);
        mbar_init(&sm.bar_mma, 1);
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
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = sm.tmem_base;
    const uint32_t lane_base = static_cast<uint32_t>(warp * 32) << 16;
    volatile int *abort_flag = &sm.abort_flag;

    const int kv_row0 = (b * p.Hkv + g) * p.S + j * kTileRows;
    if (tid == 0) {
        mbar_arrive_expect_tx(&sm.bar_kv, 2 * kTileBytes);
#pragma unroll
        for (int x = 0; x < kBoxes; ++x) {
            tma_load_2d(sm.k + x * kBoxBytesBwd, &map_k, &sm.bar_kv, x * 64, kv_row0);
            tma_load_2d(sm.v + x * kBoxBytesBwd, &map_v, &sm.bar_kv, x * 64, kv_row0);
        }
    }
    // every wait is followed by a block-wide vote so that all threads leave the loops together
    bool ok = __syncthreads_and(mbar_wait(&sm.bar_kv, 0, abort_flag, p.status, kWaitKV));

    // Power-of-two factor applied to dS before it is rounded to fp16, chosen from a bound
    // on |dS| <= |dP| + |delta| <= max||dO_row|| * max||V_row|| + max|delta| so that the scaled
    // values use fp16's normal range without overflow.  Undone exactly in the dQ/dK epilogues.
    float ds_mult = 1.f;
    if (ok) {
        float n2 = 0.f;
#pragma unroll
        for (int x = 0; x < kBoxes; ++x) {
            const uint4 *row = reinterpret_cast<const uint4 *>(sm.v + x * kBoxBytesBwd + tid * 128);
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const uint4 u = row[c];
                const __half2 *h = reinterpret_cast<const __half2 *>(&u);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float2 f = __half22float2(h[e]);
                    n2 = fmaf(f.x, f.x, n2);
                    n2 = fmaf(f.y, f.y, n2);
                }
            }
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) n2 = fmaxf(n2, __shfl_xor_sync(0xffffffffu, n2, off));
        if (lane == 0) sm.red[warp] = n2;
    }
    __syncthreads();
    {
        const float vmax2 = fmaxf(fmaxf(sm.red[0], sm.red[1]), fmaxf(sm.red[2], sm.red[3]));
        const float do2 = __uint_as_float(p.status[kStatusWordMaxDoNorm2]);
        const float dmax = __uint_as_float(p.status[kStatusWordMaxAbsDelta]);
        const float bound = sqrtf(do2) * sqrtf(vmax2) + dmax;
        int e = 24;                                  // all-zero dO: any factor works
        if (!(bound < 3.0e38f)) e = -14;             // inf/NaN inputs: outputs are non-finite anyway
        else if (bound > 1e-30f) e = min(24, max(-14, ilogbf(32768.f / bound)));
        ds_mult = ldexpf(1.f, e);
    }
    const float dq_mult = p.scale / ds_mult;
    const float scale_log2 = p.scale * kLog2e;

    const uint32_t sK = smem_u32(sm.k), sV = smem_u32(sm.v), sQ = smem_u32(sm.q), sdO = smem_u32(sm.d_o),
                   sdS = smem_u32(sm.ds);
    constexpr uint32_t idesc_s = make_idesc(128, 128, false, false);
    constexpr uint32_t idesc_dv = make_idesc(128, D, false, true);
    constexpr uint32_t idesc_dq = make_idesc(128, D, true, true);

    uint32_t phase_qdo = 0, phase_mma = 0;
    bool first = true;

    for (int hh = 0; hh < G && ok; ++hh) {
        const int h = g * G + hh;
        const long long q_head_row0 = (static_cast<long long>(b) * p.Hq + h) * p.S;
        for (int i = i_first; i < n_tiles && ok; ++i) {
            const long long q_row0 = q_head_row0 + static_cast<long long>(i) * kTileRows;
            if (tid == 0) {
                mbar_arrive_expect_tx(&sm.bar_qdo, 2 * kTileBytes);
#pragma unroll
                for (int x = 0; x < kBoxes; ++x) {
                    tma_load_2d(sm.q + x * kBoxBytesBwd, &map_q, &sm.bar_qdo, x * 64, static_cast<int>(q_row0));
                    tma_load_2d(sm.d_o + x * kBoxBytesBwd, &map_do, &sm.bar_qdo, x * 64, static_cast<int>(q_row0));
                }
            }
            sm.neg_lse_log2[tid] = -p.lse[q_row0 + tid] * kLog2e;
            sm.delta[tid] = p.delta[q_row0 + tid];
            ok = __syncthreads_and(mbar_wait(&sm.bar_qdo, phase_qdo, abort_flag, p.status, kWaitQdO));
            phase_qdo ^= 1;
            if (!ok) break;

            // S^T = K_j Q_i^T and dP^T = V_j dO_i^T
            if (tid == 0) {
                tc_fence_after_sync();
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint32_t koff = (kk >> 2) * kBoxBytesBwd + (kk & 3) * 32;
                    umma_ss(tmem + kColS, desc_kmajor(sK + koff), desc_kmajor(sQ + koff), idesc_s, kk > 0);
                }
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint32_t koff = (kk >> 2) * kBoxBytesBwd + (kk & 3) * 32;
                    umma_ss(tmem + kColdP, desc_kmajor(sV + koff), desc_kmajor(sdO + koff), idesc_s, kk > 0);
                }
                umma_commit(&sm.bar_mma);
            }
            ok = __syncthreads_and(mbar_wait(&sm.bar_mma, phase_mma, abort_flag, p.status, kWaitMma1));
            phase_mma ^= 1;
            tc_fence_after_sync();
            if (!ok) break;

            // thread = key row `tid`; columns = the 128 query rows of tile i
            uint32_t pp[64];  // P^T row as packed fp16 pairs
            const bool diag = p.causal && (i == j);
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t s[32];
                tmem_ld32(tmem + lane_base + kColS + c * 32, s);
                tmem_wait_ld();
#pragma unroll
                for (int e = 0; e < 32; e += 4) {
                    const int q0 = c * 32 + e;
                    const float4 nl = *reinterpret_cast<const float4 *>(&sm.neg_lse_log2[q0]);
                    float p0 = fast_exp2(fmaf(__uint_as_float(s[e]), scale_log2, nl.x));
                    float p1 = fast_exp2(fmaf(__uint_as_float(s[e + 1]), scale_log2, nl.y));
                    float p2 = fast_exp2(fmaf(__uint_as_float(s[e + 2]), scale_log2, nl.z));
                    float p3 = fast_exp2(fmaf(__uint_as_float(s[e + 3]), scale_log2, nl.w));
                    if (diag) {  // key row tid is hidden from query column q when tid > q
                        if (tid > q0) p0 = 0.f;
                        if (tid > q0 + 1) p1 = 0.f;
                        if (tid > q0 + 2) p2 = 0.f;
                        if (tid > q0 + 3) p3 = 0.f;
                    }
                    pp[c * 16 + e / 2] = pack_half2(p0, p1);
                    pp[c * 16 + e / 2 + 1] = pack_half2(p2, p3);
                }
                uint32_t out[16];
#pragma unroll
                for (int e = 0; e < 16; ++e) out[e] = pp[c * 16 + e];
                tmem_st16(tmem + lane_base + kColS + c * 16, out);
            }
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t dp[32];
                tmem_ld32(tmem + lane_base + kColdP + c * 32, dp);
                tmem_wait_ld();
                uint32_t o[16];
#pragma unroll
                for (int e = 0; e < 32; e += 4) {
                    const int q0 = c * 32 + e;
                    const float4 dl = *reinterpret_cast<const float4 *>(&sm.delta[q0]);
                    const float2 pa = __half22float2(*reinterpret_cast<const __half2 *>(&pp[c * 16 + e / 2]));
                    const float2 pb = __half22float2(*reinterpret_cast<const __half2 *>(&pp[c * 16 + e / 2 + 1]));
                    const float d0 = pa.x * ds_mult * (__uint_as_float(dp[e]) - dl.x);
                    const float d1 = pa.y * ds_mult * (__uint_as_float(dp[e + 1]) - dl.y);
                    const float d2 = pb.x * ds_mult * (__uint_as_float(dp[e + 2]) - dl.z);
                    const float d3 = pb.y * ds_mult * (__uint_as_float(dp[e + 3]) - dl.w);
                    o[e / 2] = pack_half2(d0, d1);
                    o[e / 2 + 1] = pack_half2(d2, d3);
                }
                // 32 query columns = four 16-byte chunks of row `tid` in tile (c / 2)
                uint8_t *tile = sm.ds + (c >> 1) * kBoxBytesBwd;
#pragma unroll
                for (int v4 = 0; v4 < 4; ++v4) {
                    const uint32_t col = (c & 1) * 32 + v4 * 8;
                    *reinterpret_cast<uint4 *>(tile + swz128_offset(tid, col)) =
                        make_uint4(o[4 * v4], o[4 * v4 + 1], o[4 * v4 + 2], o[4 * v4 + 3]);
                }
            }
            fence_proxy_async_smem();
            tmem_wait_st();
            tc_fence_before_sync();
            __syncthreads();

            if (tid == 0) {
                tc_fence_after_sync();
                const uint32_t acc0 = first ? 0u : 1u;
                // dV_j += P^T dO_i   (A = P^T from tensor memory, contraction over query rows)
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)
                    umma_ts(tmem + kColdV, tmem + kColS + kk * 8, desc_mnmajor(sdO + kk * 2048, kBoxBytesBwd),
                            idesc_dv, acc0 | (kk > 0));
                // dK_j += dS^T Q_i
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {
                    const uint32_t koff = (kk >> 2) * kBoxBytesBwd + (kk & 3) * 32;
                    umma_ss(tmem + kColdK, desc_kmajor(sdS + koff), desc_mnmajor(sQ + kk * 2048, kBoxBytesBwd),
                            idesc_dv, acc0 | (kk > 0));
                }
                // dQ_i partial = dS K_j   (contraction over key rows; overwrites the dP columns)
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)
                    umma_ss(tmem + kColdP, desc_mnmajor(sdS + kk * 2048, kBoxBytesBwd),
                            desc_mnmajor(sK + kk * 2048, kBoxBytesBwd), idesc_dq, kk > 0);
                umma_commit(&sm.bar_mma);
            }
            first = false;
            ok = __syncthreads_and(mbar_wait(&sm.bar_mma, phase_mma, abort_flag, p.status, kWaitMma2));
            phase_mma ^= 1;
            tc_fence_after_sync();
            if (!ok) break;

            // reduce the dQ partial into the fp32 accumulator: thread = query row `tid`
            float *dq_row = p.dq_acc + (q_row0 + tid) * D;
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
                uint32_t r[32];
                tmem_ld32(tmem + lane_base + kColdP + c * 32, r);
                tmem_wait_ld();
#pragma unroll
                for (int v4 = 0; v4 < 8; ++v4)
                    red_add_v4(dq_row + c * 32 + v4 * 4, __uint_as_float(r[4 * v4]) * dq_mult,
                               __uint_as_float(r[4 * v4 + 1]) * dq_mult, __uint_as_float(r[4 * v4 + 2]) * dq_mult,
                               __uint_as_float(r[4 * v4 + 3]) * dq_mult);
            }
            tc_fence_before_sync();
            __syncthreads();
        }
    }

    // epilogue: thread = key row `tid`
    if (ok && !first) {
        tc_fence_after_sync();
        __half *dk_row = p.dK + (static_cast<long long>(kv_row0) + tid) * D;
        __half *dv_row = p.dV + (static_cast<long long>(kv_row0) + tid) * D;
#pragma unroll
        for (int c = 0; c < D / 32; ++c) {
            uint32_t r[32];
            tmem_ld32(tmem + lane_base + kColdK + c * 32, r);
            tmem_wait_ld();
#pragma unroll
            for (int v8 = 0; v8 < 4; ++v8) {
                uint4 o;
                o.x = pack_half2(__uint_as_float(r[8 * v8 + 0]) * dq_mult, __uint_as_float(r[8 * v8 + 1]) * dq_mult);
                o.y = pack_half2(__uint_as_float(r[8 * v8 + 2]) * dq_mult, __uint_as_float(r[8 * v8 + 3]) * dq_mult);
                o.z = pack_half2(__uint_as_float(r[8 * v8 + 4]) * dq_mult, __uint_as_float(r[8 * v8 + 5]) * dq_mult);
                o.w = pack_half2(__uint_as_float(r[8 * v8 + 6]) * dq_mult, __uint_as_float(r[8 * v8 + 7]) * dq_mult);
                reinterpret_cast<uint4 *>(dk_row + c * 32)[v8] = o;
            }
            tmem_ld32(tmem + lane_base + kColdV + c * 32, r);
            tmem_wait_ld();
#pragma unroll
            for (int v8 = 0; v8 < 4; ++v8) {
                uint4 o;
                o.x = pack_half2(__uint_as_float(r[8 * v8 + 0]), __uint_as_float(r[8 * v8 + 1]));
                o.y = pack_half2(__uint_as_float(r[8 * v8 + 2]), __uint_as_float(r[8 * v8 + 3]));
                o.z = pack_half2(__uint_as_float(r[8 * v8 + 4]), __uint_as_float(r[8 * v8 + 5]));
                o.w = pack_half2(__uint_as_float(r[8 * v8 + 6]), __uint_as_float(r[8 * v8 + 7]));
                reinterpret_cast<uint4 *>(dv_row + c * 32)[v8] = o;
            }
        }
    }
    if (!ok && tid == 0) {
        // abandoned: give this CTA's own tile copies a bounded time to land before shared memory is released
        for (int t = 0; t < (1 << 16) && !mbar_try_wait(&sm.bar_kv, 0); ++t) {}
        for (int t = 0; t < (1 << 16) && !mbar_try_wait(&sm.bar_qdo, phase_qdo ^ 1); ++t) {}
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, kTmemCols);
}

template <int D>
static int launch_bwd(const lt_half *Q, const lt_half *K, const lt_half *V, const lt_half *O, const lt_half *dO,
                      const float *LSE, lt_half *dQ, lt_half *dK, lt_half *dV, int B, int Hq, int Hkv, int S,
                      int causal, float scale, void *workspace, cudaStream_t stream, cudaEvent_t ev_main_begin,
                      cudaEvent_t ev_main_end) {
    const long long n_rows = static_cast<long long>(B) * Hq * S;
    uint8_t *ws = static_cast<uint8_t *>(workspace);
    unsigned int *status = reinterpret_cast<unsigned int *>(ws);
    float *delta = reinterpret_cast<float *>(ws + kStatusBytes);
    float *dq_acc = reinterpret_cast<float *>(ws + kStatusBytes + round256(static_cast<size_t>(n_rows) * 4));

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
                                                             reinterpret_cast<const __half *>(O), delta, dq_acc,
                                                             n_rows, status);
    e = cudaGetLastError();
    if (e != cudaSuccess) return record_cuda_error("bwd_preprocess_kernel launch", e);

    BwdParams prm;
    prm.lse = LSE;
    prm.delta = delta;
    prm.dq_acc = dq_acc;
    prm.dK = reinterpret_cast<__half *>(dK);
    prm.dV = reinterpret_cast<__half *>(dV);
    prm.status = status;
    prm.B = B; prm.Hq = Hq; prm.Hkv = Hkv; prm.S = S; prm.causal = causal ? 1 : 0;
    prm.scale = scale;
    const size_t smem = sizeof(BwdSmem<D>) + 1024;
    e = cudaFuncSetAttribute(bwd_main_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return record_cuda_error("cudaFuncSetAttribute(bwd_main)", e);
    const int grid = B * Hkv * (S / kTileRows);
    if (ev_main_begin && (e = cudaEventRecord(ev_main_begin, stream)) != cudaSuccess)
        return record_cuda_error("cudaEventRecord", e);
    bwd_main_kernel<D><<<grid, 128, smem, stream>>>(mq, mk, mv, mdo, prm);
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
    return lt::kStatusBytes + lt::round256(n_rows * 4) + lt::round256(n_rows * D * 4);
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
