// Stand-alone microbenchmarks behind the backward kernel's bottleneck analysis (not linked into the library):
//
//   sm_limits products [reps] [grid]   cycles per tensor-core product of the main kernel's per-pair sequence
//                                      (42 products, same operand forms and tensor-memory aliasing), issued back
//                                      to back, alone and with other warps of the CTA flooding shared memory,
//                                      tensor memory, the special-function unit or the bulk-copy unit
//   sm_limits reduce [grid]            bytes per clock and SM of fp32 add-reductions into L2 (bulk and red.v4),
//                                      of plain stores and of bulk stores
//   sm_limits loadlat [grid]           latency of a 32 KB bulk load behind 0-32 KB of queued bulk reductions
//   sm_limits mixed [grid]             bulk reductions with 32 KB bulk loads running beside them (the kernel's mix)
//   sm_limits dsmem [grid]             bytes per clock and SM of stores into the partner CTA's shared memory
//                                      (clusters of two), alone and beside bulk reductions into L2
//
// Build: python -m paper_2606_10415_b200.build --microbench   (-> paper_2606_10415_b200/build/sm_limits)
// Every wait is bounded; operands are whatever the fill leaves in memory (timing does not depend on them).
#include "../lt_common.cuh"
#include <cstdio>
#include <cstdlib>
#include <cstring>
using namespace lt;

namespace {

constexpr int kBox = 128 * 128;  // one swizzled 128-row x 64-element fp16 tile
struct __align__(1024) PairSmem {
    uint8_t k[2 * kBox], v[2 * kBox], q[2][2 * kBox], d_o[2 * kBox], ds[2 * kBox];
    uint8_t ext_ones[2048], ext_q[2][2048], ext_do[2048], ext_zero[2048];
    uint64_t bar[8];
    uint32_t tmem_base;
    int stop;
};

enum Background { kNone = 0, kSmemStore, kSmemLoad, kSmemStoreConflict, kTmemLoadStore, kSfu, kBulkLoad, kBulkReduce };
const char *const kBackgroundName[] = {"none", "shared stores", "shared loads", "conflicted stores", "tensor-memory ld+st",
                                       "exponentials", "bulk loads", "bulk reductions"};

__device__ __forceinline__ uint32_t lcg(uint32_t &x) {
    x ^= x << 13; x ^= x >> 17; x ^= x << 5;
    return (x & 0x83FF83FFu) | 0x3C003C00u;  // two fp16 values in +-[1, 2)
}

// ------------------------------------------------------------------------------------------- products
// warp 1 issues `reps` times the sequence dP (9 products), dV (8, A from tensor memory), S (9), dK (8, A from
// tensor memory), dQ (8, both operands row-contracted); warps 8-15 run the background traffic.
__global__ void __launch_bounds__(512, 1)
products_kernel(int reps, int background, int random_operands, uint8_t *gmem, long long *out) {
    extern __shared__ __align__(1024) uint8_t raw[];
    PairSmem &sm = *reinterpret_cast<PairSmem *>(raw);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    gmem += static_cast<size_t>(blockIdx.x) << 20;  // 1 MB of scratch per CTA
    for (int i = tid; i < static_cast<int>(offsetof(PairSmem, bar) / 16); i += blockDim.x) {
        uint4 val = make_uint4(0, 0, 0, 0);
        if (random_operands && i < static_cast<int>(offsetof(PairSmem, ext_ones) / 16)) {
            uint32_t x = static_cast<uint32_t>(i) * 2654435761u + blockIdx.x * 40503u + 1u;
            val = make_uint4(lcg(x), lcg(x), lcg(x), lcg(x));
        }
        reinterpret_cast<uint4 *>(raw)[i] = val;
    }
    if (tid == 0) {
        for (int i = 0; i < 8; ++i) mbar_init(&sm.bar[i], 1);
        mbar_fence_init();
        sm.stop = 0;
    }
    if (warp == 0) {
        tmem_alloc(&sm.tmem_base, 512);
        tmem_relinquish();
    }
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = sm.tmem_base;
    if (random_operands && warp < 4) {
        for (int c0 = 0; c0 < 256; c0 += 16) {
            uint32_t o[16];
            uint32_t x = static_cast<uint32_t>(tid * 977 + c0) * 2654435761u + 1u;
#pragma unroll
            for (int e = 0; e < 16; ++e) o[e] = lcg(x);
            tmem_st16(tmem + (static_cast<uint32_t>(warp * 32) << 16) + c0, o);
        }
        tmem_wait_st();
        tc_fence_before_sync();
    }
    __syncthreads();
    tc_fence_after_sync();
    volatile int *stop = &sm.stop;
    constexpr uint32_t kColS = 0, kColdP = 128, kColdV = 256, kColdK = 384;
    if (warp == 1) {
        const bool leader = elect_one();
        const uint64_t wb = smem_u32(raw) >> 4;
        constexpr uint32_t oK = offsetof(PairSmem, k), oV = offsetof(PairSmem, v), oQ = offsetof(PairSmem, q);
        constexpr uint32_t oDo = offsetof(PairSmem, d_o), oDs = offsetof(PairSmem, ds), oZero = offsetof(PairSmem, ext_zero);
        constexpr uint32_t oOnes = offsetof(PairSmem, ext_ones), oExtQ = offsetof(PairSmem, ext_q), oExtDo = offsetof(PairSmem, ext_do);
        constexpr uint64_t dK_k = desc_kmajor(oK), dV_k = desc_kmajor(oV), dK_mn = desc_mnmajor(oK, kBox);
        constexpr uint64_t ddS_mn = desc_mnmajor(oDs, kBox), ddO_k = desc_kmajor(oDo), ddO_mn = desc_mnmajor(oDo, kBox);
        constexpr uint64_t dQ_k = desc_kmajor(oQ), dQ_mn = desc_mnmajor(oQ, kBox);
        constexpr uint64_t desc_ones = desc_kmajor_noswz(oOnes, oZero - oOnes, 128);
        constexpr uint64_t desc_ext_do = desc_kmajor_noswz(oExtDo, oZero - oExtDo, 128);
        constexpr uint64_t desc_ext_q = desc_kmajor_noswz(oExtQ, oZero - oExtQ, 128);
        constexpr auto koff = [](int kk) -> uint64_t { return static_cast<uint64_t>((kk >> 2) * (kBox >> 4) + (kk & 3) * 2); };
        constexpr auto roff = [](int kk) -> uint64_t { return static_cast<uint64_t>(kk * (2048 >> 4)); };
        constexpr uint32_t idesc_s = make_idesc(128, 128, false, false), idesc_dv = make_idesc(128, 128, false, true);
        constexpr uint32_t idesc_dq = make_idesc(128, 128, true, true);
        __syncwarp();
        const long long t0 = clock64();
        if (leader) {
            for (int r = 0; r < reps; ++r) {
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)  // dP^T = V dO^T
                    umma_ss(tmem + kColdP, wb + (dV_k + koff(kk)), wb + (ddO_k + koff(kk)), idesc_s, kk > 0);
                umma_ss(tmem + kColdP, wb + desc_ones, wb + desc_ext_do, idesc_s, 1);
                umma_commit(&sm.bar[0]);
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)  // dV += P'^T dO, A from the S columns
                    umma_ts(tmem + kColdV, tmem + kColS + (kk >> 2) * 64 + (kk & 3) * 8, wb + (ddO_mn + roff(kk)), idesc_dv, 1);
                umma_commit(&sm.bar[1]);
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)  // S^T = K Q^T
                    umma_ss(tmem + kColS, wb + (dK_k + koff(kk)), wb + (dQ_k + koff(kk)), idesc_s, kk > 0);
                umma_ss(tmem + kColS, wb + desc_ones, wb + desc_ext_q, idesc_s, 1);
                umma_commit(&sm.bar[2]);
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)  // dK += dS'^T Q, A from the dP columns
                    umma_ts(tmem + kColdK, tmem + kColdP + (kk >> 2) * 64 + (kk & 3) * 8, wb + (dQ_mn + roff(kk)), idesc_dv, 1);
                umma_commit(&sm.bar[3]);
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)  // dQ^T = K^T dS^T over the dP columns
                    umma_ss(tmem + kColdP, wb + (dK_mn + roff(kk)), wb + (ddS_mn + roff(kk)), idesc_dq, kk > 0);
                umma_commit(&sm.bar[4]);
            }
            umma_commit(&sm.bar[7]);
        }
        __syncwarp();
        uint32_t spins = 0;
        while (!mbar_try_wait(&sm.bar[7], 0) && ++spins < (1u << 28)) {}
        const long long t1 = clock64();
        if (lane == 0) {
            out[2 * blockIdx.x] = t1 - t0;
            *stop = 1;
        }
    } else if (warp >= 8 && background != kNone) {
        unsigned long long bytes = 0;
        uint4 acc = make_uint4(1, 2, 3, 4);
        if (background == kSmemStore || background == kSmemLoad || background == kSmemStoreConflict) {
            // 512 bytes per warp instruction; conflict-free (consecutive lanes, consecutive 16 bytes) or every lane
            // of a quarter warp on the same banks (lanes 1 KB apart)
            uint4 *base = reinterpret_cast<uint4 *>(sm.ds) +
                          (background == kSmemStoreConflict ? (warp - 8) * 8 + lane * 64 : (warp - 8) * 256 + lane);
            const int step = background == kSmemStoreConflict ? 1 : 32;
            while (!*stop) {
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    if (background == kSmemLoad) {
                        uint4 x;
                        asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                                     : "=r"(x.x), "=r"(x.y), "=r"(x.z), "=r"(x.w) : "r"(smem_u32(base + u * step)));
                        acc.x ^= x.x; acc.y ^= x.y; acc.z ^= x.z; acc.w ^= x.w;
                    } else {
                        base[u * step] = acc;
                    }
                }
                bytes += 8 * 512;
            }
        } else if (background == kTmemLoadStore) {
            // like the P pass: 32 columns read, 16 written per round (6 KB per warp)
            const uint32_t taddr = tmem + (static_cast<uint32_t>((warp & 3) * 32) << 16) + ((warp >> 2) & 1) * 64;
            while (!*stop) {
                uint32_t r[32], o[16];
                tmem_ld32(taddr, r);
                tmem_wait_ld();
#pragma unroll
                for (int e = 0; e < 16; ++e) o[e] = r[2 * e] ^ r[2 * e + 1];
                tmem_st16(taddr, o);
                tmem_wait_st();
                bytes += 6144;
            }
        } else if (background == kSfu) {
            float x[32];
#pragma unroll
            for (int e = 0; e < 32; ++e) x[e] = 0.001f * (lane + e);
            while (!*stop) {
#pragma unroll
                for (int e = 0; e < 32; ++e) x[e] = fast_exp2(fmaf(x[e], 0.5f, -1.0f));
            }
#pragma unroll
            for (int e = 0; e < 32; ++e) acc.x ^= __float_as_uint(x[e]);
        } else if (background == kBulkLoad && warp == 8 && lane == 0) {
            // 32 KB global -> shared, one at a time, like a Q or dO tile load
            uint32_t phase = 0;
            while (!*stop) {
                mbar_arrive_expect_tx(&sm.bar[6], 32768);
                bulk_load_1d(sm.q[1], gmem, 32768, &sm.bar[6]);
                uint32_t spins = 0;
                while (!mbar_try_wait(&sm.bar[6], phase) && ++spins < (1u << 24)) {}
                phase ^= 1;
                bytes += 32768;
            }
        } else if (background == kBulkReduce && warp == 8 && lane == 0) {
            // 8 KB shared -> global add.f32, two in flight, like the dQ partial
            uint32_t n = 0;
            while (!*stop) {
                bulk_reduce_add_f32(reinterpret_cast<float *>(gmem) + static_cast<size_t>(n & 63) * 2048, sm.ds, 8192);
                bulk_commit_group();
                bulk_wait_group_read<1>();
                ++n;
                bytes += 8192;
            }
            bulk_wait_group_all();
        }
        if (lane == 0 && bytes) atomicAdd(reinterpret_cast<unsigned long long *>(out + 2 * blockIdx.x + 1), bytes);
        if (acc.x == 0x12345u) out[0] = 0;  // keeps the background work alive
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, 512);
}

// ------------------------------------------------------------------------------------------- reduce
enum OutKind { kBulkRed = 0, kRedV4, kStoreV4, kBulkStore };
const char *const kOutName[] = {"cp.reduce.async.bulk add.f32", "red.global.add.v4.f32", "st.global.v4", "cp.async.bulk store"};

// One CTA per SM pushes `reps` blocks of `bytes` into its own 512 KB of L2-resident scratch.
__global__ void __launch_bounds__(128, 1) out_kernel(float *g, int bytes, int depth, int reps, int kind, long long *out) {
    extern __shared__ __align__(1024) uint8_t raw[];
    const int tid = threadIdx.x;
    for (int i = tid; i < 64 * 1024 / 4; i += blockDim.x) reinterpret_cast<float *>(raw)[i] = 1.0f;
    fence_proxy_async_smem();
    __syncthreads();
    float *dst = g + (static_cast<size_t>(blockIdx.x) << 18);  // 1 MB apart
    const int nbuf = 64 * 1024 / bytes;
    const long long t0 = clock64();
    if (kind == kBulkRed || kind == kBulkStore) {
        if (tid == 0) {
            for (int r = 0; r < reps; ++r) {
                float *d = dst + static_cast<size_t>(r % 64) * (bytes / 4) % (1 << 17);
                const uint8_t *src = raw + (r % nbuf) * bytes;
                if (kind == kBulkRed)
                    bulk_reduce_add_f32(d, src, bytes);
                else
                    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(d), "r"(smem_u32(src)), "r"(bytes) : "memory");
                bulk_commit_group();
                // at most `depth` operations in flight
                if (depth <= 1) bulk_wait_group_read<0>();
                else if (depth == 2) bulk_wait_group_read<1>();
                else if (depth <= 4) bulk_wait_group_read<3>();
                else bulk_wait_group_read<7>();
            }
            bulk_wait_group_all();
        }
    } else {
        const int per_rep = bytes / (128 * 16);  // 512 contiguous bytes per warp instruction
        for (int r = 0; r < reps; ++r)
            for (int k = 0; k < per_rep; ++k) {
                float *d = dst + (static_cast<size_t>(r % 64) * (bytes / 4) % (1 << 17)) + (k * 128 + tid) * 4;
                if (kind == kRedV4) red_add_v4(d, 1.f, 2.f, 3.f, 4.f);
                else *reinterpret_cast<float4 *>(d) = make_float4(1.f, 2.f, 3.f, 4.f);
            }
    }
    __syncthreads();
    if (tid == 0) out[blockIdx.x] = clock64() - t0;
}

// ------------------------------------------------------------------------------------------- loadlat
// Thread 0 times 32 KB bulk loads one at a time while thread 32 keeps `queued` bytes of 8 KB bulk reductions in
// flight (queued < 0: warps 2-3 issue red.v4 from registers instead).
__global__ void __launch_bounds__(128, 1) loadlat_kernel(float *g, const uint8_t *src, int queued, long long *out) {
    extern __shared__ __align__(1024) uint8_t raw[];
    __shared__ uint64_t bar;
    __shared__ int stop_flag;
    const int tid = threadIdx.x;
    for (int i = tid; i < 64 * 1024 / 4; i += blockDim.x) reinterpret_cast<float *>(raw)[i] = 1.0f;
    if (tid == 0) {
        mbar_init(&bar, 1);
        mbar_fence_init();
        stop_flag = 0;
    }
    fence_proxy_async_smem();
    __syncthreads();
    volatile int *stop = &stop_flag;
    float *dst = g + (static_cast<size_t>(blockIdx.x) << 18);
    if (tid == 0) {
        long long total = 0, worst = 0;
        for (int r = 0; r < 32; ++r) {
            for (int w = 0; w < 200; ++w) asm volatile("nanosleep.u32 50;");
            const long long t0 = clock64();
            mbar_arrive_expect_tx(&bar, 32768);
            bulk_load_1d(raw + 65536, src + (static_cast<size_t>(blockIdx.x) * 64 + r) * 32768, 32768, &bar);
            uint32_t spins = 0;
            while (!mbar_try_wait(&bar, r & 1) && ++spins < (1u << 26)) {}
            const long long dt = clock64() - t0;
            total += dt;
            worst = dt > worst ? dt : worst;
        }
        out[2 * blockIdx.x] = total / 32;
        out[2 * blockIdx.x + 1] = worst;
        *stop = 1;
    } else if (tid == 32 && queued > 0) {
        uint32_t n = 0;
        while (!*stop) {
            bulk_reduce_add_f32(dst + static_cast<size_t>(n % 16) * 2048, raw + (n % 4) * 8192, 8192);
            bulk_commit_group();
            if (queued >= 32768) bulk_wait_group_read<3>();
            else if (queued >= 16384) bulk_wait_group_read<1>();
            else bulk_wait_group_read<0>();
            ++n;
        }
        bulk_wait_group_all();
    } else if (tid >= 64 && queued < 0) {
        uint32_t n = 0;
        while (!*stop) {
            red_add_v4(dst + static_cast<size_t>(n % 256) * 256 + (tid - 64) * 4, 1.f, 2.f, 3.f, 4.f);
            ++n;
        }
    }
    __syncthreads();
}

// ------------------------------------------------------------------------------------------- dsmem
// Clusters of two CTAs: warps 0-3 of each CTA store into the partner's shared memory (16 bytes per lane, 512
// contiguous bytes per warp instruction; `with_reduce`: thread 128 issues 8 KB bulk reductions into L2 beside
// them, two in flight).  out[2*cta] = cycles, out[2*cta+1] = reduction bytes of that CTA.
__global__ void __launch_bounds__(160, 1) dsmem_kernel(float *g, int reps, int with_store, int with_reduce, long long *out) {
    extern __shared__ __align__(1024) uint8_t raw[];
    __shared__ int stop_flag;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    for (int i = tid; i < 96 * 1024 / 4; i += blockDim.x) reinterpret_cast<float *>(raw)[i] = 1.0f;
    if (tid == 0) stop_flag = 0;
    fence_proxy_async_smem();
    __syncthreads();
    cluster_sync_all();
    volatile int *stop = &stop_flag;
    const uint32_t partner = cluster_cta_rank() ^ 1u;
    float *dst = g + (static_cast<size_t>(blockIdx.x) << 18);
    const long long t0 = clock64();
    if (warp < 4) {
        if (with_store) {
            // 32 KB window of the partner, walked round and round
            const uint32_t remote = cluster_map_shared(smem_u32(raw + 32768), partner);
            for (int r = 0; r < reps; ++r) {
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const uint32_t a = remote + ((r * 4 + u) % 16) * 2048 + warp * 512 + lane * 16;
                    asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(a), "f"(1.f), "f"(2.f), "f"(3.f), "f"(4.f)
                                 : "memory");
                }
            }
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (tid == 0) {
            out[2 * blockIdx.x] = clock64() - t0;
            *stop = 1;
        }
    } else if (with_reduce && lane == 0) {
        unsigned long long bytes = 0;
        uint32_t n = 0;
        if (!with_store) {
            for (int r = 0; r < reps / 4; ++r) {  // fixed amount of work when nothing else sets the pace
                bulk_reduce_add_f32(dst + static_cast<size_t>(n & 15) * 2048, raw + (n & 3) * 8192, 8192);
                bulk_commit_group();
                bulk_wait_group_read<1>();
                ++n;
                bytes += 8192;
            }
        } else {
            while (!*stop) {
                bulk_reduce_add_f32(dst + static_cast<size_t>(n & 15) * 2048, raw + (n & 3) * 8192, 8192);
                bulk_commit_group();
                bulk_wait_group_read<1>();
                ++n;
                bytes += 8192;
            }
        }
        bulk_wait_group_all();
        out[2 * blockIdx.x + 1] = static_cast<long long>(bytes);
        if (!with_store) out[2 * blockIdx.x] = clock64() - t0;
    }
    __syncthreads();
    cluster_sync_all();  // the partner may still be storing into this CTA's shared memory
}

// ------------------------------------------------------------------------------------------- mixed
// The main kernel's own mix: thread 0 loads 32 KB tiles back to back (one at a time, as many bytes as are reduced)
// while thread 32 keeps two 8 KB bulk reductions in flight.  out[2*cta] = cycles, out[2*cta+1] = bytes loaded.
__global__ void __launch_bounds__(128, 1) mixed_kernel(float *g, const uint8_t *src, int reps, int with_loads, long long *out) {
    extern __shared__ __align__(1024) uint8_t raw[];
    __shared__ uint64_t bar;
    __shared__ int stop_flag;
    const int tid = threadIdx.x;
    for (int i = tid; i < 64 * 1024 / 4; i += blockDim.x) reinterpret_cast<float *>(raw)[i] = 1.0f;
    if (tid == 0) {
        mbar_init(&bar, 1);
        mbar_fence_init();
        stop_flag = 0;
    }
    fence_proxy_async_smem();
    __syncthreads();
    volatile int *stop = &stop_flag;
    float *dst = g + (static_cast<size_t>(blockIdx.x) << 18);
    if (tid == 32) {
        const long long t0 = clock64();
        for (int n = 0; n < reps; ++n) {
            bulk_reduce_add_f32(dst + static_cast<size_t>(n % 16) * 2048, raw + (n % 4) * 8192, 8192);
            bulk_commit_group();
            bulk_wait_group_read<1>();
        }
        bulk_wait_group_all();
        out[2 * blockIdx.x] = clock64() - t0;
        *stop = 1;
    } else if (tid == 0 && with_loads) {
        long long bytes = 0;
        uint32_t phase = 0;
        while (!*stop) {
            mbar_arrive_expect_tx(&bar, 32768);
            bulk_load_1d(raw + 65536, src + (static_cast<size_t>(blockIdx.x) * 64 + (bytes >> 15) % 64) * 32768, 32768, &bar);
            uint32_t spins = 0;
            while (!mbar_try_wait(&bar, phase) && ++spins < (1u << 26)) {}
            phase ^= 1;
            bytes += 32768;
        }
        out[2 * blockIdx.x + 1] = bytes;
    }
    __syncthreads();
}

bool check(const char *what) {
    const cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) std::printf("%s: %s\n", what, cudaGetErrorString(e));
    return e == cudaSuccess;
}

}  // namespace

int main(int argc, char **argv) {
    const char *mode = argc > 1 ? argv[1] : "products";
    long long *out;
    cudaMalloc(&out, 148 * 2 * sizeof(long long));
    if (!std::strcmp(mode, "products")) {
        const int reps = argc > 2 ? std::atoi(argv[2]) : 400, grid = argc > 3 ? std::atoi(argv[3]) : 1;
        if (grid < 1 || grid > 148) return 2;
        uint8_t *gmem;
        cudaMalloc(&gmem, static_cast<size_t>(148) << 20);
        cudaMemset(gmem, 0, static_cast<size_t>(148) << 20);
        cudaFuncSetAttribute(products_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(sizeof(PairSmem)));
        for (int random_operands = 0; random_operands <= 1; ++random_operands)
            for (int bg = kNone; bg <= kBulkReduce; ++bg) {
                if (random_operands && bg != kNone) continue;
                cudaMemset(out, 0, 148 * 2 * sizeof(long long));
                products_kernel<<<grid, 512, sizeof(PairSmem)>>>(reps, bg, random_operands, gmem, out);
                if (!check("products")) return 1;
                long long h[2];
                cudaMemcpy(h, out, sizeof(h), cudaMemcpyDeviceToHost);
                std::printf("grid %3d %s operands, background %-20s: %7.1f cycles per pair, %5.1f per product; background %6.1f B/clock\n",
                            grid, random_operands ? "random" : "zero  ", kBackgroundName[bg], static_cast<double>(h[0]) / reps,
                            static_cast<double>(h[0]) / reps / 42, static_cast<double>(h[1]) / static_cast<double>(h[0]));
            }
    } else if (!std::strcmp(mode, "reduce")) {
        const int grid = argc > 2 ? std::atoi(argv[2]) : 1, reps = 400;
        if (grid < 1 || grid > 148) return 2;
        float *g;
        cudaMalloc(&g, static_cast<size_t>(148) << 20);
        cudaMemset(g, 0, static_cast<size_t>(148) << 20);
        cudaFuncSetAttribute(out_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 64 * 1024);
        for (int kind = kBulkRed; kind <= kBulkStore; ++kind)
            for (int bytes : {4096, 8192, 16384})
                for (int depth : {1, 2, 4, 8}) {
                    if ((kind == kRedV4 || kind == kStoreV4) && depth != 1) continue;
                    if (kind == kBulkStore && depth != 2) continue;
                    for (int rep = 0; rep < 2; ++rep) out_kernel<<<grid, 128, 64 * 1024>>>(g, bytes, depth, reps, kind, out);
                    if (!check("reduce")) return 1;
                    long long h[148], worst = 0;
                    cudaMemcpy(h, out, grid * sizeof(long long), cudaMemcpyDeviceToHost);
                    for (int i = 0; i < grid; ++i) worst = h[i] > worst ? h[i] : worst;
                    std::printf("grid %3d %-30s %5d bytes, %d in flight: %7.1f cycles per block, %5.2f B/clock/SM\n", grid, kOutName[kind],
                                bytes, depth, static_cast<double>(worst) / reps, static_cast<double>(bytes) * reps / worst);
                }
    } else if (!std::strcmp(mode, "loadlat")) {
        const int grid = argc > 2 ? std::atoi(argv[2]) : 1;
        if (grid < 1 || grid > 148) return 2;
        float *g;
        uint8_t *src;
        cudaMalloc(&g, static_cast<size_t>(148) << 20);
        cudaMemset(g, 0, static_cast<size_t>(148) << 20);
        cudaMalloc(&src, static_cast<size_t>(148) * 64 * 32768);
        cudaMemset(src, 0, static_cast<size_t>(148) * 64 * 32768);
        cudaFuncSetAttribute(loadlat_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024);
        for (int queued : {0, 8192, 16384, 32768, -1}) {
            for (int rep = 0; rep < 2; ++rep) loadlat_kernel<<<grid, 128, 100 * 1024>>>(g, src, queued, out);
            if (!check("loadlat")) return 1;
            long long h[296], avg = 0, worst = 0;
            cudaMemcpy(h, out, grid * 2 * sizeof(long long), cudaMemcpyDeviceToHost);
            for (int i = 0; i < grid; ++i) {
                avg += h[2 * i];
                worst = h[2 * i + 1] > worst ? h[2 * i + 1] : worst;
            }
            if (queued >= 0)
                std::printf("grid %3d, %5d bytes of bulk reductions queued: 32 KB load latency avg %6lld, worst %6lld cycles\n", grid, queued,
                            avg / grid, worst);
            else
                std::printf("grid %3d, red.v4 from registers beside it      : 32 KB load latency avg %6lld, worst %6lld cycles\n", grid,
                            avg / grid, worst);
        }
    } else if (!std::strcmp(mode, "mixed")) {
        const int grid = argc > 2 ? std::atoi(argv[2]) : 1, reps = 2000;
        if (grid < 1 || grid > 148) return 2;
        float *g;
        uint8_t *src;
        cudaMalloc(&g, static_cast<size_t>(148) << 20);
        cudaMemset(g, 0, static_cast<size_t>(148) << 20);
        cudaMalloc(&src, static_cast<size_t>(148) * 64 * 32768);
        cudaMemset(src, 0, static_cast<size_t>(148) * 64 * 32768);
        cudaFuncSetAttribute(mixed_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024);
        for (int with_loads = 0; with_loads <= 1; ++with_loads) {
            cudaMemset(out, 0, 148 * 2 * sizeof(long long));
            for (int rep = 0; rep < 2; ++rep) mixed_kernel<<<grid, 128, 100 * 1024>>>(g, src, reps, with_loads, out);
            if (!check("mixed")) return 1;
            long long h[296], worst = 0, loaded = 0;
            cudaMemcpy(h, out, grid * 2 * sizeof(long long), cudaMemcpyDeviceToHost);
            for (int i = 0; i < grid; ++i) {
                worst = h[2 * i] > worst ? h[2 * i] : worst;
                loaded += h[2 * i + 1];
            }
            std::printf("grid %3d: bulk reductions %6.2f B/clock/SM with bulk loads of %6.2f B/clock/SM beside them\n", grid,
                        8192.0 * reps / worst, static_cast<double>(loaded) / grid / worst);
        }
    } else if (!std::strcmp(mode, "dsmem")) {
        const int grid = argc > 2 ? std::atoi(argv[2]) : 2, reps = 2000;
        if (grid < 2 || grid > 148 || (grid & 1)) return 2;
        float *g;
        cudaMalloc(&g, static_cast<size_t>(148) << 20);
        cudaMemset(g, 0, static_cast<size_t>(148) << 20);
        cudaFuncSetAttribute(dsmem_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 96 * 1024);
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(grid);
        cfg.blockDim = dim3(160);
        cfg.dynamicSmemBytes = 96 * 1024;
        cudaLaunchAttribute attr;
        attr.id = cudaLaunchAttributeClusterDimension;
        attr.val.clusterDim.x = 2;
        attr.val.clusterDim.y = 1;
        attr.val.clusterDim.z = 1;
        cfg.attrs = &attr;
        cfg.numAttrs = 1;
        const int modes[3][2] = {{1, 0}, {0, 1}, {1, 1}};
        for (auto &m : modes) {
            cudaMemset(out, 0, 148 * 2 * sizeof(long long));
            for (int rep = 0; rep < 2; ++rep)
                if (cudaLaunchKernelEx(&cfg, dsmem_kernel, g, reps, m[0], m[1], out) != cudaSuccess) {
                    std::printf("cluster launch failed: %s\n", cudaGetErrorString(cudaGetLastError()));
                    return 1;
                }
            if (!check("dsmem")) return 1;
            long long h[296], worst = 0, red = 0;
            cudaMemcpy(h, out, grid * 2 * sizeof(long long), cudaMemcpyDeviceToHost);
            for (int i = 0; i < grid; ++i) {
                worst = h[2 * i] > worst ? h[2 * i] : worst;
                red += h[2 * i + 1];
            }
            std::printf("grid %3d (clusters of 2): remote shared-memory stores %6.2f B/clock/SM, bulk reductions into L2 %6.2f B/clock/SM\n", grid,
                        m[0] ? 2048.0 * 4 * reps / worst : 0.0, static_cast<double>(red) / grid / worst);
        }
    } else {
        std::printf("usage: sm_limits products [reps] [grid] | reduce [grid] | loadlat [grid] | dsmem [grid] | mixed [grid]\n");
        return 2;
    }
    return 0;
}
