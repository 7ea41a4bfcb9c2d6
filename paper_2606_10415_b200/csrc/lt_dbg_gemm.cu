// Bring-up check of one 128x128x128 tensor-core tile product in each operand
// arrangement the attention kernels use (see lt_dbg_tile_gemm in lt_attn_debug.h).
#include "lt_common.cuh"
#include "lt_host.h"
#include "../../include/lt_attn_debug.h"

namespace lt {

constexpr int kTile = 128;
constexpr int kBoxBytes = 128 * 128;  // one swizzled tile: 128 rows x 64 fp16

struct __align__(1024) DbgSmem {
    uint8_t a[2 * kBoxBytes];
    uint8_t b[2 * kBoxBytes];
    uint8_t ext_a[2048];     // rows of (256, 1, 0, ..., 0)
    uint8_t ext_b[2048];     // rows of (hi, lo, 0, ..., 0)
    uint8_t ext_zero[2048];  // elements 8-15 of both
    uint64_t bar_load;
    uint64_t bar_mma;
    uint32_t tmem_base;
    int abort_flag;
};

__global__ void __launch_bounds__(128, 1)
dbg_tile_gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                     const __half *__restrict__ a_gmem, const __half *__restrict__ b_gmem,
                     float *__restrict__ c_gmem, int mode,
                     unsigned int *status) {
    extern __shared__ uint8_t smem_raw[];
    DbgSmem &sm = *reinterpret_cast<DbgSmem *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    constexpr uint32_t kTmemCols = 256;  // accumulator: columns 0..127, A operand: 128..191

    if (tid == 0) {
        sm.abort_flag = 0;
        mbar_init(&sm.bar_load, 1);
        mbar_init(&sm.bar_mma, 1);
        mbar_fence_init();
        tma_prefetch_desc(&map_a);
        tma_prefetch_desc(&map_b);
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

    if (tid == 0) {
        mbar_arrive_expect_tx(&sm.bar_load, 4 * kBoxBytes);
        tma_load_2d(sm.a, &map_a, &sm.bar_load, 0, 0);
        tma_load_2d(sm.a + kBoxBytes, &map_a, &sm.bar_load, 64, 0);
        tma_load_2d(sm.b, &map_b, &sm.bar_load, 0, 0);
        tma_load_2d(sm.b + kBoxBytes, &map_b, &sm.bar_load, 64, 0);
    }
    if (mode == 3) {
        // thread t owns row t of A: pack pairs of fp16 into 64 tensor-memory columns
        const uint4 *row = reinterpret_cast<const uint4 *>(a_gmem + static_cast<size_t>(tid) * kTile);
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            uint32_t r[16];
#pragma unroll
            for (int v = 0; v < 4; ++v) {
                uint4 x = row[c * 4 + v];
                r[4 * v + 0] = x.x; r[4 * v + 1] = x.y; r[4 * v + 2] = x.z; r[4 * v + 3] = x.w;
            }
            tmem_st16(tmem + lane_base + 128 + c * 16, r);
        }
        tmem_wait_st();
    }
    if (mode == 5) {
        // thread n owns row n of the two extra-step operands: adds x_n = 1000 * B[n][0] to column n
        const float x = 1000.f * __half2float(reinterpret_cast<const __half *>(b_gmem)[static_cast<size_t>(tid) * kTile]);
        const __half2 ones = __halves2half2(__float2half_rn(256.f), __float2half_rn(1.f));
        reinterpret_cast<uint4 *>(sm.ext_a)[tid] = make_uint4(*reinterpret_cast<const uint32_t *>(&ones), 0u, 0u, 0u);
        reinterpret_cast<uint4 *>(sm.ext_b)[tid] = split_ext<false>(x);
        reinterpret_cast<uint4 *>(sm.ext_zero)[tid] = make_uint4(0u, 0u, 0u, 0u);
        fence_proxy_async_smem();
    }
    tc_fence_before_sync();
    __syncthreads();

    bool ok = mbar_wait(&sm.bar_load, 0, &sm.abort_flag, status, 101);
    if (ok && tid == 0) {
        tc_fence_after_sync();
        const uint32_t a0 = smem_u32(sm.a), b0 = smem_u32(sm.b);
#pragma unroll 1
        for (int kk = 0; kk < 8; ++kk) {
            const uint32_t koff = (kk >> 2) * kBoxBytes + (kk & 3) * 32;  // contraction-contiguous operand
            const uint32_t roff = kk * 16 * 128;                          // contraction index = row
            const uint32_t acc = kk > 0;
            if (mode == 0 || mode == 4 || mode == 5 || mode == 6) {
                umma_ss(tmem, desc_kmajor(a0 + koff), desc_kmajor(b0 + koff), make_idesc(128, 128, false, false), acc);
            } else if (mode == 1) {
                umma_ss(tmem, desc_kmajor(a0 + koff), desc_mnmajor(b0 + roff, kBoxBytes),
                        make_idesc(128, 128, false, true), acc);
            } else if (mode == 2) {
                umma_ss(tmem, desc_mnmajor(a0 + roff, kBoxBytes), desc_mnmajor(b0 + roff, kBoxBytes),
                        make_idesc(128, 128, true, true), acc);
            } else {
                umma_ts(tmem, tmem + 128 + kk * 8, desc_mnmajor(b0 + roff, kBoxBytes),
                        make_idesc(128, 128, false, true), acc);
            }
        }
        if (mode == 5) {
            const uint32_t ea = smem_u32(sm.ext_a), eb = smem_u32(sm.ext_b), ez = smem_u32(sm.ext_zero);
            umma_ss(tmem, desc_kmajor_noswz(ea, ez - ea, 128), desc_kmajor_noswz(eb, ez - eb, 128),
                    make_idesc(128, 128, false, false), 1);
        }
        umma_commit(&sm.bar_mma);
    }
    ok = ok && mbar_wait(&sm.bar_mma, 0, &sm.abort_flag, status, 102);
    tc_fence_after_sync();
    // development aid: cycles for this thread to pull the 128 accumulator columns into registers
    if (ok) {
        const long long t0 = clock64();
        float acc = 0.f;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            uint32_t r[32];
            if (mode == 4) tmem_ld_16x256b_x8(tmem + (static_cast<uint32_t>(warp * 32 + (c & 1) * 16) << 16) + (c >> 1) * 64, r);
            else tmem_ld32(tmem + lane_base + c * 32, r);
            tmem_wait_ld();
#pragma unroll
            for (int e = 0; e < 32; ++e) acc += __uint_as_float(r[e]);
        }
        const long long t1 = clock64();
        if (tid == 0) {
            status[8] = static_cast<unsigned int>(t1 - t0);
            status[9] = __float_as_uint(acc);
        }
    }
    if (ok && mode == 4) {
        // read the accumulator back in the 16-lane x 256-bit arrangement the dQ reduction uses
        const int lane = tid & 31;
#pragma unroll
        for (int ch = 0; ch < 2; ++ch) {
#pragma unroll
            for (int lh = 0; lh < 2; ++lh) {
                uint32_t r[32];
                tmem_ld_16x256b_x8(tmem + (static_cast<uint32_t>(warp * 32 + lh * 16) << 16) + ch * 64, r);
                tmem_wait_ld();
                float *base = c_gmem + static_cast<size_t>(warp * 32 + lh * 16 + (lane >> 2)) * kTile + ch * 64 +
                              2 * (lane & 3);
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    *reinterpret_cast<float2 *>(base + 8 * k) =
                        make_float2(__uint_as_float(r[4 * k]), __uint_as_float(r[4 * k + 1]));
                    *reinterpret_cast<float2 *>(base + 8 * kTile + 8 * k) =
                        make_float2(__uint_as_float(r[4 * k + 2]), __uint_as_float(r[4 * k + 3]));
                }
            }
        }
    } else if (ok && mode == 6) {
        // store-arrangement probe: no product is needed; every thread writes the value
        // 1000 * row + column it believes it owns with the two 16-lane store shapes, the tile is read back
        // with the plain 32-lane shape and the host checks C[row][col] = 1000 * row + col for col < 96
        const int lane = tid & 31;
#pragma unroll
        for (int lh = 0; lh < 2; ++lh) {
            const int row0 = warp * 32 + lh * 16 + (lane >> 2);
            uint32_t r[32];
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const int col = 8 * k + 2 * (lane & 3);
                r[4 * k + 0] = __float_as_uint(1000.f * row0 + col);
                r[4 * k + 1] = __float_as_uint(1000.f * row0 + col + 1);
                r[4 * k + 2] = __float_as_uint(1000.f * (row0 + 8) + col);
                r[4 * k + 3] = __float_as_uint(1000.f * (row0 + 8) + col + 1);
            }
            tmem_st_16x256b_x8(tmem + (static_cast<uint32_t>(warp * 32 + lh * 16) << 16), r);
            uint32_t q[16];
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const int col = 64 + 4 * k + (lane & 3);
                q[2 * k + 0] = __float_as_uint(1000.f * row0 + col);
                q[2 * k + 1] = __float_as_uint(1000.f * (row0 + 8) + col);
            }
            tmem_st_16x128b_x8(tmem + (static_cast<uint32_t>(warp * 32 + lh * 16) << 16) + 64, q);
        }
        tmem_wait_st();
#pragma unroll
        for (int c = 0; c < 3; ++c) {
            uint32_t r[32];
            tmem_ld32(tmem + lane_base + c * 32, r);
            tmem_wait_ld();
            float4 *dst = reinterpret_cast<float4 *>(c_gmem + static_cast<size_t>(tid) * kTile + c * 32);
#pragma unroll
            for (int v = 0; v < 8; ++v)
                dst[v] = make_float4(__uint_as_float(r[4 * v]), __uint_as_float(r[4 * v + 1]),
                                     __uint_as_float(r[4 * v + 2]), __uint_as_float(r[4 * v + 3]));
        }
    } else if (ok) {
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            uint32_t r[32];
            tmem_ld32(tmem + lane_base + c * 32, r);
            tmem_wait_ld();
            float4 *dst = reinterpret_cast<float4 *>(c_gmem + static_cast<size_t>(tid) * kTile + c * 32);
#pragma unroll
            for (int v = 0; v < 8; ++v)
                dst[v] = make_float4(__uint_as_float(r[4 * v]), __uint_as_float(r[4 * v + 1]),
                                     __uint_as_float(r[4 * v + 2]), __uint_as_float(r[4 * v + 3]));
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, kTmemCols);
}

// A wait that nothing satisfies: exercises the bounded-wait path (no fault, no endless loop).
__global__ void dbg_wait_timeout_kernel(unsigned int *status, long long limit_cycles) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(&bar, 1);
        mbar_fence_init();
    }
    __syncthreads();
    // nobody ever arrives on `bar`; thread 0 gives up after `limit_cycles`, the others follow its flag
    const long long t0 = clock64();
    bool ok = false;
    uint32_t spins = 0;
    while (!(ok = mbar_try_wait(&bar, 0))) {
        if ((++spins & 63u) == 0u) {
            if (*reinterpret_cast<volatile int *>(&abort_flag)) break;
            if (threadIdx.x == 0 && clock64() - t0 > limit_cycles) {
                abort_flag = 1;
                atomicCAS(status + kStatusWordTimeout, 0u, 901u);
                break;
            }
        }
    }
    __syncthreads();
}

}  // namespace lt

extern "C" int lt_dbg_wait_timeout(void *workspace, size_t workspace_bytes, lt_stream_t stream) {
    using namespace lt;
    if (!workspace || !aligned256(workspace) || workspace_bytes < static_cast<size_t>(kStatusBytes))
        return LT_ERR_WORKSPACE;
    int rc = check_device();
    if (rc != LT_OK) return rc;
    cudaError_t e = cudaMemsetAsync(workspace, 0, kStatusBytes, stream);
    if (e != cudaSuccess) return record_cuda_error("cudaMemsetAsync", e);
    dbg_wait_timeout_kernel<<<1, 128, 0, stream>>>(reinterpret_cast<unsigned int *>(workspace), 20000000LL);
    e = cudaGetLastError();
    if (e != cudaSuccess) return record_cuda_error("dbg_wait_timeout_kernel launch", e);
    return LT_OK;
}

extern "C" int lt_dbg_tile_gemm(const lt_half *A, const lt_half *B, float *C, int mode, void *workspace,
                                size_t workspace_bytes, lt_stream_t stream) {
    using namespace lt;
    if (!A || !B || !C || mode < 0 || mode > 6) return LT_ERR_INVALID_ARG;
    if (!aligned16(A) || !aligned16(B) || !aligned16(C)) return LT_ERR_UNSUPPORTED;
    if (!workspace || !aligned256(workspace) || workspace_bytes < static_cast<size_t>(kStatusBytes))
        return LT_ERR_WORKSPACE;
    int rc = check_device();
    if (rc != LT_OK) return rc;
    CUtensorMap ma, mb;
    if ((rc = make_tile_map(&ma, A, 128, 128, 128)) != LT_OK) return rc;
    if ((rc = make_tile_map(&mb, B, 128, 128, 128)) != LT_OK) return rc;
    cudaError_t e = cudaMemsetAsync(workspace, 0, kStatusBytes, stream);
    if (e != cudaSuccess) return record_cuda_error("cudaMemsetAsync", e);
    const size_t smem = sizeof(DbgSmem) + 1024;
    e = cudaFuncSetAttribute(dbg_tile_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return record_cuda_error("cudaFuncSetAttribute", e);
    dbg_tile_gemm_kernel<<<1, 128, smem, stream>>>(ma, mb, reinterpret_cast<const __half *>(A),
                                                   reinterpret_cast<const __half *>(B), C, mode,
                                                   reinterpret_cast<unsigned int *>(workspace));
    e = cudaGetLastError();
    if (e != cudaSuccess) return record_cuda_error("dbg_tile_gemm_kernel launch", e);
    return LT_OK;
}
