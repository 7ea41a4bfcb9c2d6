// The paper's own forward state for Attention Backward: the probability tiles P_ij, saved by the
// forward pass and loaded by the backward instead of being recomputed (Section 4.1, the load of the
// saved tile P_ij at the top of the inner loop).  This file writes that state:
// P^T tiles, 128 keys x 128 queries of fp16 each, from Q, K and the row log-sum-exp the forward
// produced.  lt_attn_bwd_saved_p (lt_attn_bwd.cu) consumes them.
//
// Store layout: tile (b, h, j, i) - key tile j, query tile i of head h - is a 32 KB block at tile
// index ((b*Hq + h)*nT + j)*nT + i, nT = ceil(S/128).  Inside a tile, element (key, query) sits at fp16
// offset (query / 8) * 1024 + key * 8 + query % 8: sixteen blocks of eight query columns, each
// [128 keys][8 queries].  Both kernels keep one key row per thread, so with this arrangement a warp's
// 16-byte accesses are 512 contiguous bytes.
// Entries hidden by the causal mask or past the end of the sequence are zero.  Tiles wholly above
// the causal diagonal (i < j) are never read and are not written.
//
// One CTA of 128 threads per tile: TMA loads K_j and Q_i, one tensor-core product gives
// S^T = K_j Q_i^T - LSE_i/scale (the row term through the extra contraction step the backward uses),
// each thread turns one key row into probabilities and stores its sixteen 16-byte pieces.
#include "lt_common.cuh"
#include "lt_host.h"

namespace lt {

constexpr int kSpBoxBytes = 128 * 128;
constexpr float kSpLog2e = 1.4426950408889634f;
enum { kWaitSpLoad = 501, kWaitSpMma = 502 };

template <int D>
struct __align__(1024) SavePSmem {
    static constexpr int kBoxes = D / 64;
    uint8_t k[kBoxes * kSpBoxBytes];
    uint8_t q[kBoxes * kSpBoxBytes];
    uint8_t ext_ones[2048], ext_q[2048], ext_zero[2048];
    uint64_t bar_load, bar_mma;
    uint32_t tmem_base;
    int abort_flag;
};

struct SavePParams {
    const float *lse;   // [B,Hq,S]
    __half *P;          // tile store
    unsigned int *status;
    int B, Hq, Hkv, S, causal;
    float scale;
};

template <int D>
__global__ void __launch_bounds__(128, 1)
save_p_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
              const SavePParams p) {
    using Smem = SavePSmem<D>;
    constexpr int kBoxes = D / 64;
    extern __shared__ uint8_t smem_raw[];
    Smem &sm = *reinterpret_cast<Smem *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int n_tiles = (p.S + 127) / 128;
    const int i = blockIdx.x % n_tiles;
    const int j = (blockIdx.x / n_tiles) % n_tiles;
    const int bh = blockIdx.x / (n_tiles * n_tiles);
    if (p.causal && i < j) return;  // never read by the backward
    const int b = bh / p.Hq, h = bh % p.Hq;
    const int g = h / (p.Hq / p.Hkv);

    if (tid == 0) {
        sm.abort_flag = 0;
        mbar_init(&sm.bar_load, 1);
        mbar_init(&sm.bar_mma, 1);
        mbar_fence_init();
        tma_prefetch_desc(&map_q);
        tma_prefetch_desc(&map_k);
    }
    if (warp == 0) {
        tmem_alloc(&sm.tmem_base, 128);
        tmem_relinquish();
    }
    {
        // operands of the extra contraction step: multipliers, and -LSE/scale of this tile's query rows
        const uint2 mult = ext_multipliers<false>();
        const int qrow = i * 128 + tid;
        const float v = qrow < p.S ? -p.lse[static_cast<long long>(bh) * p.S + qrow] / p.scale : 0.f;
        reinterpret_cast<uint4 *>(sm.ext_ones)[tid] = make_uint4(mult.x, mult.y, 0u, 0u);
        reinterpret_cast<uint4 *>(sm.ext_q)[tid] = split_ext<false>(v);
        reinterpret_cast<uint4 *>(sm.ext_zero)[tid] = make_uint4(0u, 0u, 0u, 0u);
        fence_proxy_async_smem();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = sm.tmem_base;
    volatile int *abort_flag = &sm.abort_flag;

    if (tid == 0) {
        mbar_arrive_expect_tx(&sm.bar_load, 2 * kBoxes * kSpBoxBytes);
#pragma unroll
        for (int x = 0; x < kBoxes; ++x) {
            tma_load_4d(sm.k + x * kSpBoxBytes, &map_k, &sm.bar_load, x * 64, j * 128, g, b);
            tma_load_4d(sm.q + x * kSpBoxBytes, &map_q, &sm.bar_load, x * 64, i * 128, h, b);
        }
    }
    bool ok = __syncthreads_and(mbar_wait(&sm.bar_load, 0, abort_flag, p.status, kWaitSpLoad));
    if (ok && tid == 0) {
        tc_fence_after_sync();
        constexpr uint32_t idesc = make_idesc(128, 128, false, false);
        const uint32_t sK = smem_u32(sm.k), sQ = smem_u32(sm.q);
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
            const uint32_t koff = (kk >> 2) * kSpBoxBytes + (kk & 3) * 32;
            umma_ss(tmem, desc_kmajor(sK + koff), desc_kmajor(sQ + koff), idesc, kk > 0);
        }
        const uint32_t ez = smem_u32(sm.ext_zero), eo = smem_u32(sm.ext_ones), eq = smem_u32(sm.ext_q);
        umma_ss(tmem, desc_kmajor_noswz(eo, ez - eo, 128), desc_kmajor_noswz(eq, ez - eq, 128), idesc, 1);
        umma_commit(&sm.bar_mma);
    }
    ok = ok && __syncthreads_and(mbar_wait(&sm.bar_mma, 0, abort_flag, p.status, kWaitSpMma));
    if (ok) {
        tc_fence_after_sync();
        const int key = j * 128 + tid;  // this thread's key row
        const float scale_log2 = p.scale * kSpLog2e;
        const uint32_t lane_base = static_cast<uint32_t>(warp * 32) << 16;
        const long long tile = (static_cast<long long>(bh) * n_tiles + j) * n_tiles + i;
        // block c of a tile holds query columns 8c .. 8c+7 of all 128 key rows: [128][8] fp16
        uint4 *dst = reinterpret_cast<uint4 *>(p.P + tile * (128 * 128)) + tid;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            uint32_t r[32];
            tmem_ld32(tmem + lane_base + c * 32, r);
            tmem_wait_ld();
            uint32_t o[16];
#pragma unroll
            for (int e = 0; e < 16; ++e) {
                const int q0 = i * 128 + c * 32 + 2 * e;
                float p0 = fast_exp2(__uint_as_float(r[2 * e]) * scale_log2);
                float p1 = fast_exp2(__uint_as_float(r[2 * e + 1]) * scale_log2);
                // hidden: key after the query (causal), key or query past the end of the sequence
                if ((p.causal && key > q0) || key >= p.S || q0 >= p.S) p0 = 0.f;
                if ((p.causal && key > q0 + 1) || key >= p.S || q0 + 1 >= p.S) p1 = 0.f;
                o[e] = pack_half2(p0, p1);
            }
#pragma unroll
            for (int v4 = 0; v4 < 4; ++v4)
                dst[(c * 4 + v4) * 128] = make_uint4(o[4 * v4], o[4 * v4 + 1], o[4 * v4 + 2], o[4 * v4 + 3]);
        }
    } else if (tid == 0) {
        for (int w = 0; w < (1 << 16) && !mbar_try_wait(&sm.bar_load, 0); ++w) {}
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, 128);
}

template <int D>
static int launch_save_p(const lt_half *Q, const lt_half *K, const float *LSE, lt_half *P, int B, int Hq, int Hkv,
                         int S, int causal, float scale, void *workspace, cudaStream_t stream) {
    CUtensorMap mq, mk;
    int rc;
    if ((rc = make_bhsd_map(&mq, Q, B, Hq, S, D, contiguous_strides(Hq, S, D), 128)) != LT_OK) return rc;
    if ((rc = make_bhsd_map(&mk, K, B, Hkv, S, D, contiguous_strides(Hkv, S, D), 128)) != LT_OK) return rc;
    cudaError_t e = cudaMemsetAsync(workspace, 0, kStatusBytes, stream);
    if (e != cudaSuccess) return record_cuda_error("cudaMemsetAsync(status)", e);
    SavePParams prm;
    prm.lse = LSE;
    prm.P = reinterpret_cast<__half *>(P);
    prm.status = reinterpret_cast<unsigned int *>(workspace);
    prm.B = B; prm.Hq = Hq; prm.Hkv = Hkv; prm.S = S; prm.causal = causal ? 1 : 0;
    prm.scale = scale;
    const size_t smem = sizeof(SavePSmem<D>) + 1024;
    e = cudaFuncSetAttribute(save_p_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return record_cuda_error("cudaFuncSetAttribute(save_p)", e);
    const long long n_tiles = padded_rows(S) / 128;
    const long long grid = static_cast<long long>(B) * Hq * n_tiles * n_tiles;
    if (grid >= (1LL << 31)) return LT_ERR_UNSUPPORTED;
    save_p_kernel<D><<<static_cast<unsigned int>(grid), 128, smem, stream>>>(mq, mk, prm);
    e = cudaGetLastError();
    if (e != cudaSuccess) return record_cuda_error("save_p_kernel launch", e);
    return LT_OK;
}

}  // namespace lt

extern "C" {

size_t lt_attn_p_store_bytes(int B, int Hq, int Hkv, int S, int D) {
    if (lt::check_shape(B, Hq, Hkv, S, D, 1.0f) != LT_OK) return 0;
    const size_t n_tiles = static_cast<size_t>(lt::padded_rows(S) / 128);
    return static_cast<size_t>(B) * Hq * n_tiles * n_tiles * 128 * 128 * 2;
}

int lt_attn_save_p(const lt_half *Q, const lt_half *K, const float *LSE, lt_half *P, int B, int Hq, int Hkv, int S,
                   int D, int causal, float scale, void *workspace, size_t workspace_bytes, lt_stream_t stream) {
    using namespace lt;
    if (!Q || !K || !LSE || !P) return LT_ERR_INVALID_ARG;
    int rc = check_shape(B, Hq, Hkv, S, D, scale);
    if (rc != LT_OK) return rc;
    if (!aligned16(Q) || !aligned16(K) || !aligned256(P)) return LT_ERR_UNSUPPORTED;
    if ((reinterpret_cast<uintptr_t>(LSE) & 3u) != 0) return LT_ERR_UNSUPPORTED;
    if (!workspace || !aligned256(workspace) || workspace_bytes < kStatusBytes) return LT_ERR_WORKSPACE;
    if ((rc = check_device()) != LT_OK) return rc;
    if (D == 64) return launch_save_p<64>(Q, K, LSE, P, B, Hq, Hkv, S, causal, scale, workspace, stream);
    return launch_save_p<128>(Q, K, LSE, P, B, Hq, Hkv, S, causal, scale, workspace, stream);
}

}  // extern "C"
