// Attention forward for sm_100a: O = softmax(scale Q K^T [+ causal mask]) V and the row
// log-sum-exp.  It produces the forward state the backward needs (the paper's Algorithm 1
// takes saved probability tiles; this library keeps LSE and rebuilds P in the backward).
//
// One CTA per (batch, query head, query tile).  S = Q_i K_j^T and O += P V_j run on
// tcgen05 tensor cores; S and O live in tensor memory; each thread owns one query row
// for the online softmax.
#include "lt_common.cuh"
#include "lt_host.h"

namespace lt {

constexpr int kFwdTileRows = 128;
constexpr int kFwdBoxBytes = 128 * 128;
constexpr float kFwdLog2e = 1.4426950408889634f;
constexpr float kFwdLn2 = 0.6931471805599453f;

enum { kWaitFwdQ = 301, kWaitFwdKV = 302, kWaitFwdS = 303, kWaitFwdO = 304 };

template <int D>
struct __align__(1024) FwdSmem {
    static constexpr int kBoxes = D / 64;
    uint8_t q[kBoxes * kFwdBoxBytes];
    uint8_t k[kBoxes * kFwdBoxBytes];
    uint8_t v[kBoxes * kFwdBoxBytes];
    uint64_t bar_q, bar_kv, bar_mma;
    uint32_t tmem_base;
    int abort_flag;
};

struct FwdParams {
    __half *O;
    float *lse;
    unsigned int *status;
    int B, Hq, Hkv, S, causal;
    float scale;
};

template <int D>
__global__ void __launch_bounds__(128, 1)
fwd_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
           const __grid_constant__ CUtensorMap map_v, const FwdParams p) {
    using Smem = FwdSmem<D>;
    constexpr int kBoxes = D / 64;
    constexpr uint32_t kTileBytes = kBoxes * kFwdBoxBytes;
    constexpr uint32_t kTmemCols = 256;
    constexpr uint32_t kColS = 0, kColO = 128;

    extern __shared__ uint8_t smem_raw[];
    Smem &sm = *reinterpret_cast<Smem *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int tid = threadIdx.x;
    const int warp = tid >> 5;

    // heavy (large i) query tiles get the low block ids
    const int n_tiles = p.S / kFwdTileRows;
    const int n_bh = p.B * p.Hq;
    const int i = p.causal ? (n_tiles - 1 - blockIdx.x / n_bh) : (blockIdx.x / n_bh);
    const int bh = blockIdx.x % n_bh;
    const int b = bh / p.Hq;
    const int h = bh % p.Hq;
    const int g = h / (p.Hq / p.Hkv);
    const int j_last = p.causal ? i : n_tiles - 1;

    if (tid == 0) {
        sm.abort_flag = 0;
        mbar_init(&sm.bar_q, 1);
        mbar_init(&sm.bar_kv, 1);
        mbar_init(&sm.bar_mma, 1);
        mbar_fence_init();
        tma_prefetch_desc(&map_q);
        tma_prefetch_desc(&map_k);
        tma_prefetch_desc(&map_v);
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

    const long long q_row0 = static_cast<long long>(bh) * p.S + static_cast<long long>(i) * kFwdTileRows;
    const long long kv_head_row0 = (static_cast<long long>(b) * p.Hkv + g) * p.S;
    if (tid == 0) {
        mbar_arrive_expect_tx(&sm.bar_q, kTileBytes);
#pragma unroll
        for (int x = 0; x < kBoxes; ++x)
            tma_load_2d(sm.q + x * kFwdBoxBytes, &map_q, &sm.bar_q, x * 64, static_cast<int>(q_row0));
    }
    bool ok = __syncthreads_and(mbar_wait(&sm.bar_q, 0, abort_flag, p.status, kWaitFwdQ));

    const uint32_t sQ = smem_u32(sm.q), sK = smem_u32(sm.k), sV = smem_u32(sm.v);
    constexpr uint32_t idesc_s = make_idesc(128, 128, false, false);
    constexpr uint32_t idesc_o = make_idesc(128, D, false, true);
    const float scale_log2 = p.scale * kFwdLog2e;

    float m = -INFINITY;  // running row maximum of scale*log2(e)*score
    float l = 0.f;        // running sum of exp2(score - m)
    uint32_t phase_kv = 0, phase_mma = 0;

    for (int j = 0; j <= j_last && ok; ++j) {
        if (tid == 0) {
            const int kv_row0 = static_cast<int>(kv_head_row0 + static_cast<long long>(j) * kFwdTileRows);
            mbar_arrive_expect_tx(&sm.bar_kv, 2 * kTileBytes);
#pragma unroll
            for (int x = 0; x < kBoxes; ++x) {
                tma_load_2d(sm.k + x * kFwdBoxBytes, &map_k, &sm.bar_kv, x * 64, kv_row0);
                tma_load_2d(sm.v + x * kFwdBoxBytes, &map_v, &sm.bar_kv, x * 64, kv_row0);
            }
        }
        ok = __syncthreads_and(mbar_wait(&sm.bar_kv, phase_kv, abort_flag, p.status, kWaitFwdKV));
        phase_kv ^= 1;
        if (!ok) break;

        if (tid == 0) {
            tc_fence_after_sync();
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
                const uint32_t koff = (kk >> 2) * kFwdBoxBytes + (kk & 3) * 32;
                umma_ss(tmem + kColS, desc_kmajor(sQ + koff), desc_kmajor(sK + koff), idesc_s, kk > 0);
            }
            umma_commit(&sm.bar_mma);
        }
        ok = __syncthreads_and(mbar_wait(&sm.bar_mma, phase_mma, abort_flag, p.status, kWaitFwdS));
        phase_mma ^= 1;
        tc_fence_after_sync();
        if (!ok) break;

        // thread = query row `tid`; columns = the 128 keys of tile j
        float s[128];
        const bool diag = p.causal && (j == i);
        float row_max = -INFINITY;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            uint32_t r[32];
            tmem_ld32(tmem + lane_base + kColS + c * 32, r);
            tmem_wait_ld();
#pragma unroll
            for (int e = 0; e < 32; ++e) {
                float x = __uint_as_float(r[e]) * scale_log2;
                if (diag && (c * 32 + e) > tid) x = -INFINITY;
                s[c * 32 + e] = x;
                row_max = fmaxf(row_max, x);
            }
        }
        const float m_new = fmaxf(m, row_max);
        const float alpha = fast_exp2(m - m_new);  // 0 on the first tile (m = -inf)
        float row_sum = 0.f;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            uint32_t out[16];
#pragma unroll
            for (int e = 0; e < 32; e += 2) {
                const float p0 = fast_exp2(s[c * 32 + e] - m_new);
                const float p1 = fast_exp2(s[c * 32 + e + 1] - m_new);
                // sum the values the tensor core will see (fp16-rounded) so that O / l is consistent
                const __half2 hp = __floats2half2_rn(p0, p1);
                const float2 back = __half22float2(hp);
                row_sum += back.x + back.y;
                out[e / 2] = *reinterpret_cast<const uint32_t *>(&hp);
            }
            tmem_st16(tmem + lane_base + kColS + c * 16, out);
        }
        l = l * alpha + row_sum;
        m = m_new;
        if (j > 0) {
            // rescale the running output
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
                uint32_t r[32];
                tmem_ld32(tmem + lane_base + kColO + c * 32, r);
                tmem_wait_ld();
#pragma unroll
                for (int e = 0; e < 32; ++e) r[e] = __float_as_uint(__uint_as_float(r[e]) * alpha);
                tmem_st32(tmem + lane_base + kColO + c * 32, r);
            }
        }
        tmem_wait_st();
        tc_fence_before_sync();
        __syncthreads();

        if (tid == 0) {
            tc_fence_after_sync();
            // O += P V_j   (A = P from tensor memory, contraction over the key rows of V)
#pragma unroll
            for (int kk = 0; kk < 8; ++kk)
                umma_ts(tmem + kColO, tmem + kColS + kk * 8, desc_mnmajor(sV + kk * 2048, kFwdBoxBytes), idesc_o,
                        (j > 0) | (kk > 0));
            umma_commit(&sm.bar_mma);
        }
        ok = __syncthreads_and(mbar_wait(&sm.bar_mma, phase_mma, abort_flag, p.status, kWaitFwdO));
        phase_mma ^= 1;
        tc_fence_after_sync();
    }

    if (ok) {
        const float inv_l = 1.f / l;
        __half *o_row = p.O + (q_row0 + tid) * D;
#pragma unroll
        for (int c = 0; c < D / 32; ++c) {
            uint32_t r[32];
            tmem_ld32(tmem + lane_base + kColO + c * 32, r);
            tmem_wait_ld();
#pragma unroll
            for (int v8 = 0; v8 < 4; ++v8) {
                uint4 o;
                o.x = pack_half2(__uint_as_float(r[8 * v8 + 0]) * inv_l, __uint_as_float(r[8 * v8 + 1]) * inv_l);
                o.y = pack_half2(__uint_as_float(r[8 * v8 + 2]) * inv_l, __uint_as_float(r[8 * v8 + 3]) * inv_l);
                o.z = pack_half2(__uint_as_float(r[8 * v8 + 4]) * inv_l, __uint_as_float(r[8 * v8 + 5]) * inv_l);
                o.w = pack_half2(__uint_as_float(r[8 * v8 + 6]) * inv_l, __uint_as_float(r[8 * v8 + 7]) * inv_l);
                reinterpret_cast<uint4 *>(o_row + c * 32)[v8] = o;
            }
        }
        p.lse[q_row0 + tid] = (m + log2f(l)) * kFwdLn2;
    } else if (tid == 0) {
        for (int t = 0; t < (1 << 16) && !mbar_try_wait(&sm.bar_q, 0); ++t) {}
        for (int t = 0; t < (1 << 16) && !mbar_try_wait(&sm.bar_kv, phase_kv ^ 1); ++t) {}
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, kTmemCols);
}

template <int D>
static int launch_fwd(const lt_half *Q, const lt_half *K, const lt_half *V, lt_half *O, float *LSE, int B, int Hq,
                      int Hkv, int S, int causal, float scale, void *workspace, cudaStream_t stream) {
    CUtensorMap mq, mk, mv;
    int rc;
    if ((rc = make_tile_map(&mq, Q, static_cast<uint64_t>(B) * Hq * S, D, 128)) != LT_OK) return rc;
    if ((rc = make_tile_map(&mk, K, static_cast<uint64_t>(B) * Hkv * S, D, 128)) != LT_OK) return rc;
    if ((rc = make_tile_map(&mv, V, static_cast<uint64_t>(B) * Hkv * S, D, 128)) != LT_OK) return rc;
    cudaError_t e = cudaMemsetAsync(workspace, 0, kStatusBytes, stream);
    if (e != cudaSuccess) return record_cuda_error("cudaMemsetAsync(status)", e);
    FwdParams prm;
    prm.O = reinterpret_cast<__half *>(O);
    prm.lse = LSE;
    prm.status = reinterpret_cast<unsigned int *>(workspace);
    prm.B = B; prm.Hq = Hq; prm.Hkv = Hkv; prm.S = S; prm.causal = causal ? 1 : 0;
    prm.scale = scale;
    const size_t smem = sizeof(FwdSmem<D>) + 1024;
    e = cudaFuncSetAttribute(fwd_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return record_cuda_error("cudaFuncSetAttribute(fwd)", e);
    const int grid = B * Hq * (S / kFwdTileRows);
    fwd_kernel<D><<<grid, 128, smem, stream>>>(mq, mk, mv, prm);
    e = cudaGetLastError();
    if (e != cudaSuccess) return record_cuda_error("fwd_kernel launch", e);
    return LT_OK;
}

}  // namespace lt

extern "C" {

size_t lt_attn_fwd_workspace_bytes(int B, int Hq, int Hkv, int S, int D) {
    if (lt::check_shape(B, Hq, Hkv, S, D, 1.0f) != LT_OK) return 0;
    return lt::kStatusBytes;
}

int lt_attn_fwd_num_launches(void) { return 1; }

int lt_attn_fwd(const lt_half *Q, const lt_half *K, const lt_half *V, lt_half *O, float *LSE, int B, int Hq, int Hkv,
                int S, int D, int causal, float scale, void *workspace, size_t workspace_bytes, lt_stream_t stream) {
    using namespace lt;
    if (!Q || !K || !V || !O || !LSE) return LT_ERR_INVALID_ARG;
    int rc = check_shape(B, Hq, Hkv, S, D, scale);
    if (rc != LT_OK) return rc;
    const void *ptrs[] = {Q, K, V, O, LSE};
    for (const void *ptr : ptrs)
        if (!aligned16(ptr)) return LT_ERR_UNSUPPORTED;
    if (!workspace || !aligned256(workspace) || workspace_bytes < lt_attn_fwd_workspace_bytes(B, Hq, Hkv, S, D))
        return LT_ERR_WORKSPACE;
    if ((rc = check_device()) != LT_OK) return rc;
    if (D == 64) return launch_fwd<64>(Q, K, V, O, LSE, B, Hq, Hkv, S, causal, scale, workspace, stream);
    return launch_fwd<128>(Q, K, V, O, LSE, B, Hq, Hkv, S, causal, scale, workspace, stream);
}

size_t lt_attn_host_arena_bytes(int B, int Hq, int Hkv, int S, int D) {
    const size_t wb = lt_attn_bwd_workspace_bytes(B, Hq, Hkv, S, D);
    if (wb == 0) return 0;
    const size_t nq = lt::round256(static_cast<size_t>(B) * Hq * S * D * 2);
    const size_t nk = lt::round256(static_cast<size_t>(B) * Hkv * S * D * 2);
    const size_t nl = lt::round256(static_cast<size_t>(B) * Hq * S * 4);
    // Q, dO, O, dQ | K, V, dK, dV | LSE | forward status block | backward workspace
    return 4 * nq + 4 * nk + nl + lt::kStatusBytes + wb;
}

int lt_attn_fwd_bwd_host(const lt_half *Q, const lt_half *K, const lt_half *V, const lt_half *dO, lt_half *O,
                         float *LSE, lt_half *dQ, lt_half *dK, lt_half *dV, int B, int Hq, int Hkv, int S, int D,
                         int causal, float scale, void *arena, size_t arena_bytes, lt_stream_t stream) {
    using namespace lt;
    if (!Q || !K || !V || !dO || !dQ || !dK || !dV) return LT_ERR_INVALID_ARG;
    int rc = check_shape(B, Hq, Hkv, S, D, scale);
    if (rc != LT_OK) return rc;
    const size_t need = lt_attn_host_arena_bytes(B, Hq, Hkv, S, D);
    if (!arena || !aligned256(arena) || arena_bytes < need) return LT_ERR_WORKSPACE;
    const size_t bq = static_cast<size_t>(B) * Hq * S * D * 2, bk = static_cast<size_t>(B) * Hkv * S * D * 2;
    const size_t bl = static_cast<size_t>(B) * Hq * S * 4;
    const size_t nq = round256(bq), nk = round256(bk), nl = round256(bl);
    uint8_t *a = static_cast<uint8_t *>(arena);
    lt_half *d_Q = reinterpret_cast<lt_half *>(a);
    lt_half *d_dO = reinterpret_cast<lt_half *>(a + nq);
    lt_half *d_O = reinterpret_cast<lt_half *>(a + 2 * nq);
    lt_half *d_dQ = reinterpret_cast<lt_half *>(a + 3 * nq);
    uint8_t *kbase = a + 4 * nq;
    lt_half *d_K = reinterpret_cast<lt_half *>(kbase);
    lt_half *d_V = reinterpret_cast<lt_half *>(kbase + nk);
    lt_half *d_dK = reinterpret_cast<lt_half *>(kbase + 2 * nk);
    lt_half *d_dV = reinterpret_cast<lt_half *>(kbase + 3 * nk);
    float *d_lse = reinterpret_cast<float *>(kbase + 4 * nk);
    void *fwd_ws = kbase + 4 * nk + nl;
    void *ws = kbase + 4 * nk + nl + kStatusBytes;
    const size_t ws_bytes = arena_bytes - (4 * nq + 4 * nk + nl + kStatusBytes);

    cudaError_t e;
#define LT_COPY(dst, src, n, kind)                                                       \
    if ((e = cudaMemcpyAsync(dst, src, n, kind, stream)) != cudaSuccess)                 \
        return record_cuda_error("cudaMemcpyAsync", e)
    LT_COPY(d_Q, Q, bq, cudaMemcpyHostToDevice);
    LT_COPY(d_K, K, bk, cudaMemcpyHostToDevice);
    LT_COPY(d_V, V, bk, cudaMemcpyHostToDevice);
    LT_COPY(d_dO, dO, bq, cudaMemcpyHostToDevice);
    rc = lt_attn_fwd(d_Q, d_K, d_V, d_O, d_lse, B, Hq, Hkv, S, D, causal, scale, fwd_ws, kStatusBytes, stream);
    if (rc != LT_OK) return rc;
    rc = lt_attn_bwd(d_Q, d_K, d_V, d_O, d_dO, d_lse, d_dQ, d_dK, d_dV, B, Hq, Hkv, S, D, causal, scale, ws,
                     ws_bytes, stream);
    if (rc != LT_OK) return rc;
    if (O) LT_COPY(O, d_O, bq, cudaMemcpyDeviceToHost);
    if (LSE) LT_COPY(LSE, d_lse, bl, cudaMemcpyDeviceToHost);
    LT_COPY(dQ, d_dQ, bq, cudaMemcpyDeviceToHost);
    LT_COPY(dK, d_dK, bk, cudaMemcpyDeviceToHost);
    LT_COPY(dV, d_dV, bk, cudaMemcpyDeviceToHost);
#undef LT_COPY
    return LT_OK;
}

}  // extern "C"
