// FP16 GEMM for sm_100a: C[M,N] = A[M,K] W[N,K]^T, fp16 operands, fp32 accumulation, fp16 result.
// This is the linear-layer primitive of the paper's backend (Section 4.1, "FP16 GEMM assembly
// pipeline"; shapes profiled in Section 6.6).  The MT-3000 dataflow of the paper (A staged through
// GSM/SM, B broadcast to AM, C accumulated in AM) maps here to: A and W tiles staged in shared memory
// by TMA, C accumulated in tensor memory, one CTA per SM walking the output tiles.
//
//   warp 0      : TMA producer - 64-wide contraction blocks of a 128-row A tile and a 256-row W
//                 tile through a four-slot ring
//   warp 1      : tcgen05 issuer - four 128x256x16 products per block into one of two 256-column
//                 accumulators
//   warps 2..5  : epilogue - tensor memory -> fp16 -> global, one accumulator while the other is
//                 being filled
#include <cstdlib>
#include "lt_common.cuh"
#include "lt_host.h"

namespace lt {

constexpr int kGemmBM = 128, kGemmBN = 256, kGemmBK = 64, kGemmStages = 4;
constexpr int kGemmThreads = 192;
constexpr uint32_t kGemmABytes = kGemmBM * kGemmBK * 2;   // 16 KB
constexpr uint32_t kGemmBBytes = kGemmBN * kGemmBK * 2;   // 32 KB

enum { kWaitGemmFull = 401, kWaitGemmEmpty = 402, kWaitGemmAccFull = 403, kWaitGemmAccEmpty = 404 };

struct __align__(1024) GemmSmem {
    uint8_t a[kGemmStages][kGemmABytes];
    uint8_t b[kGemmStages][kGemmBBytes];
    uint64_t bar_full[kGemmStages], bar_empty[kGemmStages], bar_acc_full[2], bar_acc_empty[2];
    uint32_t tmem_base;
    int abort_flag;
};

struct GemmParams {
    __half *C;
    unsigned int *status;
    int M, N, K;
    int tiles_m, tiles_n;
    int group_rows;  // tile rows of A kept hot in L2 while the W column blocks stream past them
};

// Output tiles are numbered so that consecutive numbers share the W tile (the larger operand tile)
// and a wave of CTAs covers a compact block of C: tile -> (m, n) with m fastest inside groups of
// `group_rows` tile rows (as many rows of A as stay resident in L2, so that W is read from DRAM once
// per group).
__device__ __forceinline__ void gemm_tile_coords(const GemmParams &p, int tile, int &tm, int &tn) {
    const int kGroup = p.group_rows;
    const int per_group = kGroup * p.tiles_n;
    const int g = tile / per_group;
    const int first_m = g * kGroup;
    const int rows = min(kGroup, p.tiles_m - first_m);
    const int r = tile - g * per_group;
    tm = first_m + r % rows;
    tn = r / rows;
}

template <bool kBf16>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
            const GemmParams p) {
    extern __shared__ uint8_t smem_raw[];
    GemmSmem &sm = *reinterpret_cast<GemmSmem *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;
    const int n_tiles = p.tiles_m * p.tiles_n;
    const int k_blocks = (p.K + kGemmBK - 1) / kGemmBK;  // a ragged last block reads zeros past K

    if (tid == 0) {
        sm.abort_flag = 0;
        for (int s = 0; s < kGemmStages; ++s) {
            mbar_init(&sm.bar_full[s], 1);
            mbar_init(&sm.bar_empty[s], 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(&sm.bar_acc_full[a], 1);
            mbar_init(&sm.bar_acc_empty[a], 4);  // lane 0 of each epilogue warp
        }
        mbar_fence_init();
        tma_prefetch_desc(&map_a);
        tma_prefetch_desc(&map_b);
    }
    if (warp == 0) {
        tmem_alloc(&sm.tmem_base, 512);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = sm.tmem_base;
    volatile int *abort_flag = &sm.abort_flag;

    if (warp == 0) {
        if (lane == 0) {
            bool ok = true;
            int kb_total = 0;  // contraction blocks loaded so far, over all tiles
            for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
                int tm, tn;
                gemm_tile_coords(p, tile, tm, tn);
                for (int kb = 0; kb < k_blocks; ++kb, ++kb_total) {
                    const int s = kb_total % kGemmStages;
                    const uint32_t use = kb_total / kGemmStages;
                    if (use >= 1 && !(ok = mbar_wait(&sm.bar_empty[s], (use - 1) & 1, abort_flag, p.status, kWaitGemmEmpty)))
                        break;
                    mbar_arrive_expect_tx(&sm.bar_full[s], kGemmABytes + kGemmBBytes);
                    tma_load_2d(sm.a[s], &map_a, &sm.bar_full[s], kb * kGemmBK, tm * kGemmBM);
                    tma_load_2d(sm.b[s], &map_b, &sm.bar_full[s], kb * kGemmBK, tn * kGemmBN);
                }
            }
            if (!ok || *abort_flag) {
                // somebody gave up: wait (bounded) for the copies in flight before the CTA exits
                for (int back = 0; back < kGemmStages && back < kb_total; ++back) {
                    const int q = kb_total - 1 - back;
                    for (int w = 0; w < (1 << 16) && !mbar_try_wait(&sm.bar_full[q % kGemmStages], (q / kGemmStages) & 1); ++w) {}
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc(kGemmBM, kGemmBN, false, false, kBf16);
            bool ok = true;
            int kb_total = 0, t_local = 0;
#ifdef LT_GEMM_TRACE
            long long tr_full = 0, tr_acc = 0, tr_issue = 0, tr_t = clock64();
#define LT_GT(var) do { const long long n_ = clock64(); var += n_ - tr_t; tr_t = n_; } while (0)
#else
#define LT_GT(var)
#endif
            for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++t_local) {
                const int acc = t_local & 1;
                const uint32_t acc_use = t_local >> 1;
                // the epilogue must have read this accumulator's previous tile
                if (acc_use >= 1 && !(ok = mbar_wait(&sm.bar_acc_empty[acc], (acc_use - 1) & 1, abort_flag, p.status, kWaitGemmAccEmpty)))
                    break;
                LT_GT(tr_acc);
                tc_fence_after_sync();
                for (int kb = 0; kb < k_blocks; ++kb, ++kb_total) {
                    const int s = kb_total % kGemmStages;
                    LT_GT(tr_issue);
                    if (!(ok = mbar_wait(&sm.bar_full[s], (kb_total / kGemmStages) & 1, abort_flag, p.status, kWaitGemmFull))) break;
                    LT_GT(tr_full);
                    tc_fence_after_sync();
                    const uint64_t da = desc_kmajor(smem_u32(sm.a[s])), db = desc_kmajor(smem_u32(sm.b[s]));
#pragma unroll
                    for (int kk = 0; kk < kGemmBK / 16; ++kk)
                        umma_ss(tmem + acc * kGemmBN, da + kk * 2, db + kk * 2, idesc, (kb > 0) | (kk > 0));
                    umma_commit(&sm.bar_empty[s]);  // the slot is free once these products have read it
                }
                if (!ok) break;
                umma_commit(&sm.bar_acc_full[acc]);
                LT_GT(tr_issue);
            }
#ifdef LT_GEMM_TRACE
            if (blockIdx.x == 0) {
                p.status[8] = static_cast<unsigned int>(tr_full >> 4);
                p.status[9] = static_cast<unsigned int>(tr_acc >> 4);
                p.status[10] = static_cast<unsigned int>(tr_issue >> 4);
                p.status[11] = static_cast<unsigned int>(kb_total);
            }
#endif
        }
    } else {
        // epilogue: thread = row of the tile, 32 columns at a time
        const int quad = warp & 3;  // tensor-memory lane quadrant this warp may read
        const int row = quad * 32 + lane;
        const uint32_t lane_base = static_cast<uint32_t>(quad * 32) << 16;
        bool ok = true;
        int t_local = 0;
        for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++t_local) {
            const int acc = t_local & 1;
            ok = mbar_wait(&sm.bar_acc_full[acc], (t_local >> 1) & 1, abort_flag, p.status, kWaitGemmAccFull);
            if (!(ok = __all_sync(0xffffffffu, ok))) break;
            tc_fence_after_sync();
            int tm, tn;
            gemm_tile_coords(p, tile, tm, tn);
            const long long m = static_cast<long long>(tm) * kGemmBM + row;
            const int n0 = tn * kGemmBN;
            __half *c_row = p.C + m * p.N + n0;
            const bool vec_ok = (p.N % 8) == 0;  // 16-byte stores need the row pitch to allow them
#pragma unroll
            for (int c = 0; c < kGemmBN / 32; ++c) {
                uint32_t r[32];
                tmem_ld32(tmem + lane_base + acc * kGemmBN + c * 32, r);
                tmem_wait_ld();
                if (c == kGemmBN / 32 - 1) {
                    // the whole accumulator is in registers or stored: the issuer may reuse it
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&sm.bar_acc_empty[acc]);
                }
                if (m < p.M) {
                    const int nc = n0 + c * 32;
                    if (vec_ok && nc + 32 <= p.N) {
#pragma unroll
                        for (int v8 = 0; v8 < 4; ++v8) {
                            uint4 o;
                            o.x = pack2<kBf16>(__uint_as_float(r[8 * v8 + 0]), __uint_as_float(r[8 * v8 + 1]));
                            o.y = pack2<kBf16>(__uint_as_float(r[8 * v8 + 2]), __uint_as_float(r[8 * v8 + 3]));
                            o.z = pack2<kBf16>(__uint_as_float(r[8 * v8 + 4]), __uint_as_float(r[8 * v8 + 5]));
                            o.w = pack2<kBf16>(__uint_as_float(r[8 * v8 + 6]), __uint_as_float(r[8 * v8 + 7]));
                            reinterpret_cast<uint4 *>(c_row + c * 32)[v8] = o;
                        }
                    } else {
#pragma unroll
                        for (int e = 0; e < 32; ++e)
                            if (nc + e < p.N)
                                reinterpret_cast<uint16_t *>(c_row)[c * 32 + e] =
                                    static_cast<uint16_t>(pack2<kBf16>(__uint_as_float(r[e]), 0.f) & 0xFFFFu);
                    }
                }
            }
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, 512);
}

// ----------------------------------------------------------------------------- CTA-pair variant
// Two CTAs of a cluster work one 256 x 256 output tile: each loads 128 rows of A and 128 of the 256 rows of
// W per contraction block (32 KB per block and CTA where the single-CTA kernel loads 48 KB for the same
// number of FLOPs per SM), the even CTA issues 256x256x16 pair products, and each CTA's epilogue stores the
// 128 rows of C that its tensor memory holds.  Barriers: `full` lives in the issuing CTA and collects the
// bytes of both CTAs' loads; `empty` and `acc_full` are signalled in both CTAs by pair commits; `acc_empty`
// lives in the issuing CTA and is arrived on by the epilogue warps of both.
constexpr int kPairBM = 256, kPairBN = 256, kPairStages = 6;
constexpr uint32_t kPairABytes = 128 * kGemmBK * 2;   // 16 KB: this CTA's rows of the A tile
constexpr uint32_t kPairBBytes = 128 * kGemmBK * 2;   // 16 KB: this CTA's half of the W tile's rows

struct __align__(1024) GemmPairSmem {
    uint8_t a[kPairStages][kPairABytes];
    uint8_t b[kPairStages][kPairBBytes];
    uint64_t bar_full[kPairStages], bar_empty[kPairStages], bar_acc_full[2], bar_acc_empty[2];
    uint32_t tmem_base;
    int abort_flag;
};

template <bool kBf16>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kGemmThreads, 1)
gemm_pair_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                 const GemmParams p) {
    extern __shared__ uint8_t smem_raw[];
    // (the dynamic window starts at the same offset in both CTAs, so the aligned structure does too)
    GemmPairSmem &sm =
        *reinterpret_cast<GemmPairSmem *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;
    const uint32_t rank = cluster_cta_rank();   // 0 issues the products
    const int pair = blockIdx.x >> 1;
    const int n_pairs = gridDim.x >> 1;
    const int n_tiles = p.tiles_m * p.tiles_n;  // 256 x 256 tiles
    const int k_blocks = (p.K + kGemmBK - 1) / kGemmBK;

    if (tid == 0) {
        sm.abort_flag = 0;
        for (int s = 0; s < kPairStages; ++s) {
            mbar_init(&sm.bar_full[s], 1);
            mbar_init(&sm.bar_empty[s], 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(&sm.bar_acc_full[a], 1);
            mbar_init(&sm.bar_acc_empty[a], 8);  // lane 0 of each epilogue warp of both CTAs
        }
        mbar_fence_init();
        tma_prefetch_desc(&map_a);
        tma_prefetch_desc(&map_b);
    }
    if (warp == 0) {
        tmem_alloc_pair(&sm.tmem_base, 512);
        tmem_relinquish_pair();
    }
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync_all();  // the partner's barriers exist before anything is sent to them
    tc_fence_after_sync();
    const uint32_t tmem = sm.tmem_base;
    volatile int *abort_flag = &sm.abort_flag;

    if (warp == 0) {
        if (lane == 0) {
            bool ok = true;
            int kb_total = 0;
            for (int tile = pair; tile < n_tiles && ok; tile += n_pairs) {
                int tm, tn;
                gemm_tile_coords(p, tile, tm, tn);
                const int a_row = tm * kPairBM + static_cast<int>(rank) * 128;
                const int b_row = tn * kPairBN + static_cast<int>(rank) * 128;
                for (int kb = 0; kb < k_blocks; ++kb, ++kb_total) {
                    const int s = kb_total % kPairStages;
                    const uint32_t use = kb_total / kPairStages;
                    if (use >= 1 && !(ok = mbar_wait(&sm.bar_empty[s], (use - 1) & 1, abort_flag, p.status, kWaitGemmEmpty)))
                        break;
                    // the issuing CTA's barrier expects the bytes of all four loads of the pair
                    if (rank == 0) mbar_arrive_expect_tx(&sm.bar_full[s], 2 * (kPairABytes + kPairBBytes));
                    const uint32_t full0 = cluster_map_shared(smem_u32(&sm.bar_full[s]), 0);
                    tma_load_2d_pair(sm.a[s], &map_a, full0, kb * kGemmBK, a_row);
                    tma_load_2d_pair(sm.b[s], &map_b, full0, kb * kGemmBK, b_row);
                }
            }
            if (!ok || *abort_flag) {
                // somebody gave up: give this CTA's own copies a bounded time to land (the slots' `empty`
                // barriers cannot tell; the issuing CTA's `full` barriers can, for the last slots used)
                if (rank == 0)
                    for (int back = 0; back < kPairStages && back < kb_total; ++back) {
                        const int q = kb_total - 1 - back;
                        for (int w = 0; w < (1 << 16) && !mbar_try_wait(&sm.bar_full[q % kPairStages], (q / kPairStages) & 1); ++w) {}
                    }
                else
                    for (int w = 0; w < 256; ++w) __nanosleep(100);  // (its byte counts go to the partner's barriers)
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {
            constexpr uint32_t idesc = make_idesc(kPairBM, kPairBN, false, false, kBf16);
            bool ok = true;
            int kb_total = 0, t_local = 0;
            for (int tile = pair; tile < n_tiles && ok; tile += n_pairs, ++t_local) {
                const int acc = t_local & 1;
                const uint32_t acc_use = t_local >> 1;
                if (acc_use >= 1 && !(ok = mbar_wait(&sm.bar_acc_empty[acc], (acc_use - 1) & 1, abort_flag, p.status, kWaitGemmAccEmpty)))
                    break;
                tc_fence_after_sync();
                for (int kb = 0; kb < k_blocks; ++kb, ++kb_total) {
                    const int s = kb_total % kPairStages;
                    if (!(ok = mbar_wait(&sm.bar_full[s], (kb_total / kPairStages) & 1, abort_flag, p.status, kWaitGemmFull))) break;
                    tc_fence_after_sync();
                    const uint64_t da = desc_kmajor(smem_u32(sm.a[s])), db = desc_kmajor(smem_u32(sm.b[s]));
#pragma unroll
                    for (int kk = 0; kk < kGemmBK / 16; ++kk)
                        umma_ss_pair(tmem + acc * kPairBN, da + kk * 2, db + kk * 2, idesc, (kb > 0) | (kk > 0));
                    umma_commit_pair(&sm.bar_empty[s], 3);  // both CTAs' slots are free once these have read them
                }
                if (!ok) break;
                umma_commit_pair(&sm.bar_acc_full[acc], 3);
            }
        }
    } else {
        // epilogue: this CTA's 128 rows of the tile; thread = row, 32 columns at a time
        const int quad = warp & 3;
        const int row = quad * 32 + lane;
        const uint32_t lane_base = static_cast<uint32_t>(quad * 32) << 16;
        bool ok = true;
        int t_local = 0;
        for (int tile = pair; tile < n_tiles; tile += n_pairs, ++t_local) {
            const int acc = t_local & 1;
            ok = mbar_wait(&sm.bar_acc_full[acc], (t_local >> 1) & 1, abort_flag, p.status, kWaitGemmAccFull);
            if (!(ok = __all_sync(0xffffffffu, ok))) break;
            tc_fence_after_sync();
            int tm, tn;
            gemm_tile_coords(p, tile, tm, tn);
            const long long m = static_cast<long long>(tm) * kPairBM + rank * 128 + row;
            const int n0 = tn * kPairBN;
            __half *c_row = p.C + m * p.N + n0;
            const bool vec_ok = (p.N % 8) == 0;
            const uint32_t acc_empty0 = cluster_map_shared(smem_u32(&sm.bar_acc_empty[acc]), 0);
#pragma unroll
            for (int c = 0; c < kPairBN / 32; ++c) {
                uint32_t r[32];
                tmem_ld32(tmem + lane_base + acc * kPairBN + c * 32, r);
                tmem_wait_ld();
                if (c == kPairBN / 32 - 1) {
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive_cluster(acc_empty0);
                }
                if (m < p.M) {
                    const int nc = n0 + c * 32;
                    if (vec_ok && nc + 32 <= p.N) {
#pragma unroll
                        for (int v8 = 0; v8 < 4; ++v8) {
                            uint4 o;
                            o.x = pack2<kBf16>(__uint_as_float(r[8 * v8 + 0]), __uint_as_float(r[8 * v8 + 1]));
                            o.y = pack2<kBf16>(__uint_as_float(r[8 * v8 + 2]), __uint_as_float(r[8 * v8 + 3]));
                            o.z = pack2<kBf16>(__uint_as_float(r[8 * v8 + 4]), __uint_as_float(r[8 * v8 + 5]));
                            o.w = pack2<kBf16>(__uint_as_float(r[8 * v8 + 6]), __uint_as_float(r[8 * v8 + 7]));
                            reinterpret_cast<uint4 *>(c_row + c * 32)[v8] = o;
                        }
                    } else {
#pragma unroll
                        for (int e = 0; e < 32; ++e)
                            if (nc + e < p.N)
                                reinterpret_cast<uint16_t *>(c_row)[c * 32 + e] =
                                    static_cast<uint16_t>(pack2<kBf16>(__uint_as_float(r[e]), 0.f) & 0xFFFFu);
                    }
                }
            }
        }
    }

    // neither CTA may release its tensor memory or leave (its shared memory and barriers are still
    // targets of the partner) before both are done
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync_all();
    if (warp == 0) tmem_dealloc_pair(tmem, 512);
}

}  // namespace lt

extern "C" {

size_t lt_gemm_f16_workspace_bytes(void) { return lt::kStatusBytes; }

static int gemm_entry(const void *A, const void *W, void *C, int M, int N, int K, void *workspace,
                      size_t workspace_bytes, lt_stream_t stream, bool bf16) {
    using namespace lt;
    if (!A || !W || !C) return LT_ERR_INVALID_ARG;
    if (M <= 0 || N <= 0 || K <= 0) return LT_ERR_INVALID_ARG;
    // TMA needs 16-byte row pitches for the operands
    if ((K % 8) != 0) return LT_ERR_UNSUPPORTED;
    if (!aligned16(A) || !aligned16(W) || !aligned16(C)) return LT_ERR_UNSUPPORTED;
    if (!workspace || !aligned256(workspace) || workspace_bytes < kStatusBytes) return LT_ERR_WORKSPACE;
    int rc = check_device();
    if (rc != LT_OK) return rc;

    // More than one 128-row tile of A: CTA pairs work 256 x 256 tiles (LT_GEMM_SINGLE_CTA=1 in the
    // environment keeps the single-CTA kernel, for comparison).
    static const bool force_single = [] {
        const char *v = getenv("LT_GEMM_SINGLE_CTA");
        return v && v[0] == '1';
    }();
    const bool use_pair = M > kGemmBM && !force_single;

    CUtensorMap ma, mb;
    if ((rc = make_tile_map(&ma, A, M, K, kGemmBM)) != LT_OK) return rc;
    if ((rc = make_tile_map(&mb, W, N, K, use_pair ? 128 : kGemmBN)) != LT_OK) return rc;
    cudaError_t e = cudaMemsetAsync(workspace, 0, kStatusBytes, stream);
    if (e != cudaSuccess) return record_cuda_error("cudaMemsetAsync(status)", e);
    if (use_pair) {
        GemmParams prm;
        prm.C = reinterpret_cast<__half *>(C);
        prm.status = reinterpret_cast<unsigned int *>(workspace);
        prm.M = M; prm.N = N; prm.K = K;
        prm.tiles_m = (M + kPairBM - 1) / kPairBM;
        prm.tiles_n = (N + kPairBN - 1) / kPairBN;
        const long long rows = static_cast<long long>(48.0e6 / (static_cast<double>(kPairBM) * K * 2.0));
        prm.group_rows = static_cast<int>(rows < 1 ? 1 : (rows > prm.tiles_m ? prm.tiles_m : rows));
        const size_t smem = sizeof(GemmPairSmem) + 1024;
        auto kernel = bf16 ? gemm_pair_kernel<true> : gemm_pair_kernel<false>;
        e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
        if (e != cudaSuccess) return record_cuda_error("cudaFuncSetAttribute(gemm_pair)", e);
        // CTA pairs that can be resident at once (every pair needs two SMs of one cluster-capable group)
        static int max_pairs_cached[2] = {0, 0};
        int &max_pairs = max_pairs_cached[bf16 ? 1 : 0];
        if (max_pairs == 0) {
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3(2);
            cfg.blockDim = dim3(kGemmThreads);
            cfg.dynamicSmemBytes = smem;
            cudaLaunchAttribute attr;
            attr.id = cudaLaunchAttributeClusterDimension;
            attr.val.clusterDim.x = 2;
            attr.val.clusterDim.y = 1;
            attr.val.clusterDim.z = 1;
            cfg.attrs = &attr;
            cfg.numAttrs = 1;
            int n = 0;
            e = cudaOccupancyMaxActiveClusters(&n, kernel, &cfg);
            if (e != cudaSuccess || n < 1) return record_cuda_error("cudaOccupancyMaxActiveClusters", e);
            max_pairs = n;
        }
        const long long n_tiles = static_cast<long long>(prm.tiles_m) * prm.tiles_n;
        const int pairs = static_cast<int>(n_tiles < max_pairs ? n_tiles : max_pairs);
        kernel<<<2 * pairs, kGemmThreads, smem, stream>>>(ma, mb, prm);
        e = cudaGetLastError();
        if (e != cudaSuccess) return record_cuda_error("gemm_pair_kernel launch", e);
        return LT_OK;
    }

    GemmParams prm;
    prm.C = reinterpret_cast<__half *>(C);
    prm.status = reinterpret_cast<unsigned int *>(workspace);
    prm.M = M; prm.N = N; prm.K = K;
    prm.tiles_m = (M + kGemmBM - 1) / kGemmBM;
    prm.tiles_n = (N + kGemmBN - 1) / kGemmBN;
    {
        // about 48 MB of A rows per group (L2 holds 126 MB; the rest is for the W blocks in flight and C)
        const long long rows = static_cast<long long>(48.0e6 / (static_cast<double>(kGemmBM) * K * 2.0));
        prm.group_rows = static_cast<int>(rows < 1 ? 1 : (rows > prm.tiles_m ? prm.tiles_m : rows));
    }
    const size_t smem = sizeof(GemmSmem) + 1024;
    auto kernel = bf16 ? gemm_kernel<true> : gemm_kernel<false>;
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return record_cuda_error("cudaFuncSetAttribute(gemm)", e);
    int sms = 148;
    {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    }
    const long long n_tiles = static_cast<long long>(prm.tiles_m) * prm.tiles_n;
    const int grid = static_cast<int>(n_tiles < sms ? n_tiles : sms);
    kernel<<<grid, kGemmThreads, smem, stream>>>(ma, mb, prm);
    e = cudaGetLastError();
    if (e != cudaSuccess) return record_cuda_error("gemm_kernel launch", e);
    return LT_OK;
}

int lt_gemm_f16(const lt_half *A, const lt_half *W, lt_half *C, int M, int N, int K, void *workspace,
                size_t workspace_bytes, lt_stream_t stream) {
    return gemm_entry(A, W, C, M, N, K, workspace, workspace_bytes, stream, false);
}

int lt_gemm_bf16(const lt_bf16 *A, const lt_bf16 *W, lt_bf16 *C, int M, int N, int K, void *workspace,
                 size_t workspace_bytes, lt_stream_t stream) {
    return gemm_entry(A, W, C, M, N, K, workspace, workspace_bytes, stream, true);
}

}  // extern "C"
