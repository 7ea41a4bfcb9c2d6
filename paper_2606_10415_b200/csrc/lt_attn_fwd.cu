// Attention forward for sm_100a: O = softmax(scale Q K^T [+ causal mask]) V and the row
// log-sum-exp.  It produces the forward state the backward needs (the paper's Algorithm 1
// takes saved probability tiles; this library keeps LSE and rebuilds P in the backward).
//
// One CTA per (batch, query head, pair of neighbouring 128-row query tiles).  Warp 0 streams
// K_j / V_j tiles with TMA through two-stage rings, warp 1 issues S = Q_i K_j^T and
// O += P V_j on the tcgen05 tensor cores, and each query tile has its own group of four
// softmax warps (one thread per query row), so that the tensor cores work on one tile of the
// pair while the other tile's scores are exponentiated.  S/P and O live in tensor memory.
// The running row maximum is only raised when it grew by more than 2^8 since the output
// was last rescaled, so most key tiles need no pass over O.
#include <algorithm>
#include <mutex>
#include <type_traits>

#include "lt_common.cuh"
#include "lt_host.h"

namespace lt {

constexpr int kFwdTileRows = 128;
constexpr int kFwdBoxBytes = 128 * 128;
constexpr float kFwdLog2e = 1.4426950408889634f;
constexpr float kFwdLn2 = 0.6931471805599453f;
// three warpgroups: control (producer warp, issuer warp, two warps that only fill up the group) and 2 x 4
// softmax warps; the control group hands most of its registers to the softmax warps, each of whose threads
// keeps the 128 scores of a query row in registers
constexpr int kFwdThreads = 384;
constexpr int kFwdSoftmaxWarp0 = 4;
constexpr int kFwdRegsAtLaunch = 168, kFwdRegsControl = 80, kFwdRegsSoftmax = 208;
static_assert(kFwdRegsAtLaunch * kFwdThreads <= 65536 && 128 * kFwdRegsControl + 256 * kFwdRegsSoftmax <= 65536,
              "register shares exceed the register file");
constexpr float kFwdRescaleLog2 = 8.f;        // P <= 2^8 stays far inside fp16 range

enum {
    kWaitFwdQ = 301, kWaitFwdK = 302, kWaitFwdV = 303, kWaitFwdS = 304, kWaitFwdP = 305,
    kWaitFwdO = 306, kWaitFwdKEmpty = 307, kWaitFwdVEmpty = 308, kWaitFwdDone = 309
};

template <int D>
struct __align__(1024) FwdSmem {
    static constexpr int kBoxes = D / 64;
    static constexpr int kTile = kBoxes * kFwdBoxBytes;
    uint8_t q[2][kTile];   // the pair's two query tiles
    uint8_t k[2][kTile];   // ring of key tiles
    uint8_t v[2][kTile];   // ring of value tiles
    uint64_t bar_q[2], bar_k_full[2], bar_k_empty[2], bar_v_full[2], bar_v_empty[2];
    uint64_t bar_s_full[2], bar_p_ready[2], bar_p_half[2], bar_o_done[2], bar_done;
    uint32_t tmem_base;
    int abort_flag;
};

struct FwdParams {
    __half *O;
    float *lse;
    unsigned int *status;
    int B, Hq, Hkv, S, causal;
    float scale;
    lt_tensor_strides o_st;  // element strides of O
};

#ifdef LT_FWD_TRACE
// Development build only: summed clock() intervals.  [0..7] issuer, [8..15] softmax lane 0 of
// every warp, [16] tiles processed by softmax warps, [17] key tiles seen by issuers, [18] CTA cycles.
__device__ unsigned long long g_fwd_trace[32];
#define LT_FT_DECL uint32_t ft_acc[8] = {0, 0, 0, 0, 0, 0, 0, 0}; uint32_t ft_t = clock()
#define LT_FT(slot) do { const uint32_t ft_n = clock(); ft_acc[slot] += ft_n - ft_t; ft_t = ft_n; } while (0)
#define LT_FT_FLUSH(base) do { for (int ft_i = 0; ft_i < 8; ++ft_i) if (ft_acc[ft_i]) atomicAdd(&g_fwd_trace[(base) + ft_i], static_cast<unsigned long long>(ft_acc[ft_i])); } while (0)
#define LT_FT_COUNT(slot, n) atomicAdd(&g_fwd_trace[slot], static_cast<unsigned long long>(n))
#else
#define LT_FT_DECL
#define LT_FT(slot)
#define LT_FT_FLUSH(base)
#define LT_FT_COUNT(slot, n)
#endif

// Registers are handed out per four warps, so ten warps get the 168-register cap of twelve.
template <int D, bool kBf16>
__global__ void __launch_bounds__(kFwdThreads, 1)
fwd_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
           const __grid_constant__ CUtensorMap map_v, const FwdParams p) {
    using Smem = FwdSmem<D>;
    constexpr int kBoxes = D / 64;
    constexpr uint32_t kTileBytes = Smem::kTile;
    constexpr uint32_t kTmemCols = 512;
    constexpr uint32_t kColS = 0;     // tile t: S / P at columns [128 t, 128 t + 128)
    constexpr uint32_t kColO = 256;   // tile t: O at columns [256 + D t, 256 + D t + D)

    extern __shared__ uint8_t smem_raw[];
    Smem &sm = *reinterpret_cast<Smem *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;

    // heavy (late) query-tile pairs get the low block ids
    const int n_tiles = (p.S + kFwdTileRows - 1) / kFwdTileRows;  // the last tile may be ragged
    const int n_pairs = (n_tiles + 1) / 2;
    const int n_bh = p.B * p.Hq;
    const int pr = p.causal ? (n_pairs - 1 - blockIdx.x / n_bh) : (blockIdx.x / n_bh);
    const int bh = blockIdx.x % n_bh;
    const int b = bh / p.Hq;
    const int h = bh % p.Hq;
    const int g = h / (p.Hq / p.Hkv);
    const int i0 = 2 * pr;
    const bool has_b = (i0 + 1) < n_tiles;
    // last key tile of query tile t; -1 when the pair has no second tile
    const int j_last0 = p.causal ? i0 : n_tiles - 1;
    const int j_last1 = has_b ? (p.causal ? i0 + 1 : n_tiles - 1) : -1;
    const int j_end = j_last0 > j_last1 ? j_last0 : j_last1;

    if (tid == 0) {
        sm.abort_flag = 0;
#pragma unroll
        for (int t = 0; t < 2; ++t) {
            mbar_init(&sm.bar_q[t], 1);
            mbar_init(&sm.bar_k_full[t], 1);
            mbar_init(&sm.bar_k_empty[t], 1);
            mbar_init(&sm.bar_v_full[t], 1);
            mbar_init(&sm.bar_v_empty[t], 1);
            mbar_init(&sm.bar_s_full[t], 1);
            mbar_init(&sm.bar_p_ready[t], 128);
            mbar_init(&sm.bar_p_half[t], 128);
            mbar_init(&sm.bar_o_done[t], 1);
        }
        mbar_init(&sm.bar_done, 1);
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
    volatile int *abort_flag = &sm.abort_flag;


    if (warp < kFwdSoftmaxWarp0) {
        warpgroup_regs_set<kFwdRegsControl, kFwdRegsAtLaunch>();
        if (warp == 0) {
            // ------------------------------------------------------------------ producer
            if (lane == 0) {
                for (int t = 0; t < (has_b ? 2 : 1); ++t) {
                    mbar_arrive_expect_tx(&sm.bar_q[t], kTileBytes);
#pragma unroll
                    for (int x = 0; x < kBoxes; ++x)
                        tma_load_4d(sm.q[t] + x * kFwdBoxBytes, &map_q, &sm.bar_q[t], x * 64, (i0 + t) * kFwdTileRows, h, b);
                }
                bool ok = true;
                int armed = 0;  // key/value tiles whose loads were started
                for (int j = 0; j <= j_end; ++j) {
                    const int s = j & 1;
                    const uint32_t ph = (j >> 1) & 1;
                    const int kv_row0 = j * kFwdTileRows;  // inside the head; rows past S arrive as zeros
                    if (j >= 2 && !(ok = mbar_wait(&sm.bar_k_empty[s], ph ^ 1, abort_flag, p.status, kWaitFwdKEmpty))) break;
                    mbar_arrive_expect_tx(&sm.bar_k_full[s], kTileBytes);
#pragma unroll
                    for (int x = 0; x < kBoxes; ++x)
                        tma_load_4d(sm.k[s] + x * kFwdBoxBytes, &map_k, &sm.bar_k_full[s], x * 64, kv_row0, g, b);
                    if (j >= 2 && !(ok = mbar_wait(&sm.bar_v_empty[s], ph ^ 1, abort_flag, p.status, kWaitFwdVEmpty))) {
                        // the key tile just started still has to land before shared memory is given up
                        for (int w = 0; w < (1 << 16) && !mbar_try_wait(&sm.bar_k_full[s], ph); ++w) {}
                        break;
                    }
                    mbar_arrive_expect_tx(&sm.bar_v_full[s], kTileBytes);
#pragma unroll
                    for (int x = 0; x < kBoxes; ++x)
                        tma_load_4d(sm.v[s] + x * kFwdBoxBytes, &map_v, &sm.bar_v_full[s], x * 64, kv_row0, g, b);
                    armed = j + 1;
                }
                if (!ok || *abort_flag) {
                    // somebody gave up: wait (bounded) for the copies in flight before the CTA exits
                    for (int t = 0; t < (has_b ? 2 : 1); ++t)
                        for (int w = 0; w < (1 << 16) && !mbar_try_wait(&sm.bar_q[t], 0); ++w) {}
                    for (int j = armed > 2 ? armed - 2 : 0; j < armed; ++j) {
                        for (int w = 0; w < (1 << 16) && !mbar_try_wait(&sm.bar_k_full[j & 1], (j >> 1) & 1); ++w) {}
                        for (int w = 0; w < (1 << 16) && !mbar_try_wait(&sm.bar_v_full[j & 1], (j >> 1) & 1); ++w) {}
                    }
                }
            }
        } else if (warp == 1) {
            // ------------------------------------------------------------------ MMA issuer
            // The whole warp walks the loop, so that counters, wait results (voted) and descriptor arithmetic are
            // warp-uniform; one elected lane issues the products and commits.
            {
                const bool leader = elect_one();
                auto wait_all = [&](uint64_t *bar, uint32_t parity, int code) {
                    return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag, p.status, code));
                };
                // descriptors of slot 0; slot 1 of each ring follows one tile later
                const uint64_t dQ0 = desc_kmajor(smem_u32(sm.q[0])), dK0 = desc_kmajor(smem_u32(sm.k[0]));
                const uint64_t dV0 = desc_mnmajor(smem_u32(sm.v[0]), kFwdBoxBytes);
                constexpr uint64_t kSlotStep = static_cast<uint64_t>(kTileBytes) >> 4;
                auto koff = [](int kk) -> uint64_t { return static_cast<uint64_t>((kk >> 2) * (kFwdBoxBytes >> 4) + (kk & 3) * 2); };
                auto roff = [](int kk) -> uint64_t { return static_cast<uint64_t>(kk * (2048 >> 4)); };
                constexpr uint32_t idesc_s = make_idesc(128, 128, false, false, kBf16);
                constexpr uint32_t idesc_o = make_idesc(128, D, false, true, kBf16);
                auto issue_s = [&](int t, int s) {  // S_t = Q_t K^T with the key tile in ring slot s
                    if (!leader) return;
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk)
                        umma_ss(tmem + kColS + t * 128, dQ0 + t * kSlotStep + koff(kk), dK0 + s * kSlotStep + koff(kk), idesc_s, kk > 0);
                    umma_commit(&sm.bar_s_full[t]);
                };
                // O_t (+)= P_t V, P_t read from tensor memory; the keys of a tile in two halves of 64, so that the
                // first half's products run while the softmax warps exponentiate the second half (quarters were
                // measured too and lost to the extra hand-offs)
                auto issue_pv_half = [&](int t, int s, bool acc, int half) {
                    if (!leader) return;
#pragma unroll
                    for (int kk = 4 * half; kk < 4 * half + 4; ++kk)
                        umma_ts(tmem + kColO + t * D, tmem + kColS + t * 128 + kk * 8, dV0 + s * kSlotStep + roff(kk), idesc_o,
                                acc | (kk > 0));
                    if (half == 1) umma_commit(&sm.bar_o_done[t]);
                };
                bool ok = wait_all(&sm.bar_q[0], 0, kWaitFwdQ) &&
                          (!has_b || wait_all(&sm.bar_q[1], 0, kWaitFwdQ)) &&
                          wait_all(&sm.bar_k_full[0], 0, kWaitFwdK);
                if (ok) {
                    tc_fence_after_sync();
                    issue_s(0, 0);
                    if (has_b) issue_s(1, 0);
                    if (leader) umma_commit(&sm.bar_k_empty[0]);
                }
                LT_FT_DECL;
                for (int j = 0; j <= j_end && ok; ++j) {
                    const int s = j & 1, sn = s ^ 1;
                    LT_FT(0);
                    if (!(ok = wait_all(&sm.bar_v_full[s], (j >> 1) & 1, kWaitFwdV))) break;
                    LT_FT(1);
                    bool k_next_ready = false;
#pragma unroll
                    for (int t = 0; t < 2; ++t) {
                        const int j_last_t = t == 0 ? j_last0 : j_last1;
                        if (j > j_last_t) continue;
                        LT_FT(0);
                        if (!(ok = wait_all(&sm.bar_p_half[t], j & 1, kWaitFwdP))) break;
                        tc_fence_after_sync();
                        issue_pv_half(t, s, j > 0, 0);
                        if (!(ok = wait_all(&sm.bar_p_ready[t], j & 1, kWaitFwdP))) break;
                        LT_FT(2 + t);
                        tc_fence_after_sync();
                        LT_FT(0);
                        issue_pv_half(t, s, j > 0, 1);
                        LT_FT(5);
                        // the second tile of the pair, when it uses this key tile, uses it last
                        const int last_user = (j <= j_last1) ? 1 : 0;
                        if (t == last_user && leader) umma_commit(&sm.bar_v_empty[s]);
                        if (j + 1 <= j_last_t) {
                            if (!k_next_ready) {
                                LT_FT(0);
                                if (!(ok = wait_all(&sm.bar_k_full[sn], ((j + 1) >> 1) & 1, kWaitFwdK))) break;
                                LT_FT(4);
                                tc_fence_after_sync();
                                k_next_ready = true;
                            }
                            LT_FT(0);
                            issue_s(t, sn);
                            LT_FT(6);
                            const int last_user_next = (j + 1 <= j_last1) ? 1 : 0;
                            if (t == last_user_next && leader) umma_commit(&sm.bar_k_empty[sn]);
                        }
                    }
                }
                LT_FT(0);
                LT_FT_FLUSH(0);
                LT_FT_COUNT(17, j_end + 1);
                // every product issued above has finished before tensor memory is released
                if (leader) umma_commit(&sm.bar_done);
                if (!wait_all(&sm.bar_done, 0, kWaitFwdDone))
                    for (int w = 0; w < (1 << 16) && !mbar_try_wait(&sm.bar_done, 0); ++w) {}
            }
        }
    } else {
        // ------------------------------------------------------------------ softmax warps
        warpgroup_regs_set<kFwdRegsSoftmax, kFwdRegsAtLaunch>();
        const int t = (warp - kFwdSoftmaxWarp0) >> 2;   // which query tile of the pair
        const int quad = warp & 3;                      // tensor-memory lane quadrant of this warp
        const int row = quad * 32 + lane;               // query row inside the tile
        const int j_last = t == 0 ? j_last0 : j_last1;
        const int i = i0 + t;
        const uint32_t lane_base = static_cast<uint32_t>(quad * 32) << 16;
        const uint32_t tS = tmem + lane_base + kColS + t * 128;
        const uint32_t tO = tmem + lane_base + kColO + t * D;
        const float scale_log2 = p.scale * kFwdLog2e;
        // last visible key of a masked tile: the row's own index on a causal diagonal tile, the end of
        // the sequence on the ragged last key tile without a causal mask
        const int tail_keys = p.S - (n_tiles - 1) * kFwdTileRows;
        const int last_key = p.causal ? row : tail_keys - 1;
        float m_used = -INFINITY;  // the maximum the stored P, l and O are relative to
        float l = 0.f;             // running sum of exp2(score - m_used)
        bool ok = true;
        LT_FT_DECL;
        for (int j = 0; j <= j_last; ++j) {
            LT_FT(0);
            ok = mbar_wait(&sm.bar_s_full[t], j & 1, abort_flag, p.status, kWaitFwdS);
            LT_FT(1);
            if (!(ok = __all_sync(0xffffffffu, ok))) break;
            tc_fence_after_sync();
            // the whole score row of this key tile stays in registers
            uint32_t sc[128];
#pragma unroll
            for (int c = 0; c < 4; ++c) tmem_ld32(tS + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&sc[c * 32]));
            tmem_wait_ld();
            LT_FT(2);
            float rs[4] = {0.f, 0.f, 0.f, 0.f};  // independent partial row sums
            auto tile_softmax = [&](auto diag_tag) {
                constexpr bool kMasked = decltype(diag_tag)::value;  // keys past `last_key` are invisible
                // row extremum of the raw scores over the unmasked keys: the maximum of
                // scale*log2(e)*score is that factor times the largest (smallest, for a negative
                // scale) raw score
                // (eight independent running extrema: one warp per scheduler has no other work to
                // cover the latency of a dependent chain)
                float ex[8];
                if (scale_log2 >= 0.f) {
#pragma unroll
                    for (int u = 0; u < 8; ++u) ex[u] = -INFINITY;
#pragma unroll
                    for (int e = 0; e < 64; ++e) {  // two keys per step: a three-input maximum
                        const float a = (!kMasked || e <= last_key) ? __uint_as_float(sc[e]) : -INFINITY;
                        const float c = (!kMasked || e + 64 <= last_key) ? __uint_as_float(sc[e + 64]) : -INFINITY;
                        ex[e & 7] = fmaxf(ex[e & 7], fmaxf(a, c));
                    }
#pragma unroll
                    for (int u = 4; u > 0; u >>= 1)
#pragma unroll
                        for (int w = 0; w < u; ++w) ex[w] = fmaxf(ex[w], ex[w + u]);
                } else {
#pragma unroll
                    for (int u = 0; u < 8; ++u) ex[u] = INFINITY;
#pragma unroll
                    for (int e = 0; e < 64; ++e) {
                        const float a = (!kMasked || e <= last_key) ? __uint_as_float(sc[e]) : INFINITY;
                        const float c = (!kMasked || e + 64 <= last_key) ? __uint_as_float(sc[e + 64]) : INFINITY;
                        ex[e & 7] = fminf(ex[e & 7], fminf(a, c));
                    }
#pragma unroll
                    for (int u = 4; u > 0; u >>= 1)
#pragma unroll
                        for (int w = 0; w < u; ++w) ex[w] = fminf(ex[w], ex[w + u]);
                }
                const float ext = ex[0];
                const float row_max = ext * scale_log2;
                LT_FT(3);
                if (j == 0) {
                    m_used = row_max;  // key 0 is never masked, so this is finite for finite inputs
                } else {
                    const bool raise = (row_max - m_used) > kFwdRescaleLog2;
                    if (__any_sync(0xffffffffu, raise)) {
                        // O must hold every earlier product before it is rescaled
                        ok = mbar_wait(&sm.bar_o_done[t], (j - 1) & 1, abort_flag, p.status, kWaitFwdO);
                        if (!(ok = __all_sync(0xffffffffu, ok))) return;
                        tc_fence_after_sync();
                        const float alpha = raise ? fast_exp2(m_used - row_max) : 1.f;
#pragma unroll
                        for (int c = 0; c < D / 16; ++c) {  // narrow pieces: the score row holds most registers
                            uint32_t r[16];
                            tmem_ld16(tO + c * 16, r);
                            tmem_wait_ld();
#pragma unroll
                            for (int e = 0; e < 16; ++e) r[e] = __float_as_uint(__uint_as_float(r[e]) * alpha);
                            tmem_st16(tO + c * 16, r);
                        }
                        l *= alpha;
                        if (raise) m_used = row_max;
                    }
                }
                LT_FT(4);
                // P = exp2(score - m_used) as fp16 over the first 64 columns of the S region
                const float neg_m = -m_used;
#pragma unroll
                for (int half = 0; half < 2; ++half) {
#pragma unroll
                    for (int e = 64 * half; e < 64 * half + 64; ++e) {
                        const float x = fmaf(__uint_as_float(sc[e]), scale_log2, neg_m);
                        float pe = fast_exp2(x);
                        if (kMasked && e > last_key) pe = 0.f;
                        rs[e & 3] += pe;
                        sc[e] = __float_as_uint(pe);
                    }
#pragma unroll
                    for (int c = 2 * half; c < 2 * half + 2; ++c) {
                        uint32_t out[16];
#pragma unroll
                        for (int e = 0; e < 32; e += 2)
                            out[e / 2] = pack2<kBf16>(__uint_as_float(sc[c * 32 + e]), __uint_as_float(sc[c * 32 + e + 1]));
                        tmem_st16(tS + c * 16, out);
                    }
                    if (half == 0) {
                        // the first 64 keys' probabilities are in place: their products may start
                        tmem_wait_st();
                        tc_fence_before_sync();
                        mbar_arrive(&sm.bar_p_half[t]);
                    }
                }
            };
            if (p.causal ? (j == i) : (j == n_tiles - 1 && tail_keys < kFwdTileRows)) tile_softmax(std::true_type{});
            else tile_softmax(std::false_type{});
            if (!ok) break;
            const float row_sum = (rs[0] + rs[1]) + (rs[2] + rs[3]);
            l += row_sum;
            LT_FT(5);
            tmem_wait_st();
            tc_fence_before_sync();
            mbar_arrive(&sm.bar_p_ready[t]);
            LT_FT(6);
        }
#ifdef LT_FWD_TRACE
        if (lane == 0) {
            LT_FT_FLUSH(8);
            LT_FT_COUNT(16, j_last + 1);
        }
#endif

        if (ok && j_last >= 0) {
            ok = mbar_wait(&sm.bar_o_done[t], j_last & 1, abort_flag, p.status, kWaitFwdO);
            ok = __all_sync(0xffffffffu, ok);
        }
        if (ok && j_last >= 0) {
            tc_fence_after_sync();
            const float inv_l = 1.f / l;
            const int s_row = i * kFwdTileRows + row;  // rows past S belong to nobody
            const long long q_row = static_cast<long long>(bh) * p.S + s_row;  // LSE is contiguous
            __half *o_row = p.O + b * p.o_st.batch + h * p.o_st.head + s_row * p.o_st.row;
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
                uint32_t r[32];
                tmem_ld32(tO + c * 32, r);
                tmem_wait_ld();
#pragma unroll
                for (int v8 = 0; v8 < 4; ++v8) {
                    uint4 o;
                    o.x = pack2<kBf16>(__uint_as_float(r[8 * v8 + 0]) * inv_l, __uint_as_float(r[8 * v8 + 1]) * inv_l);
                    o.y = pack2<kBf16>(__uint_as_float(r[8 * v8 + 2]) * inv_l, __uint_as_float(r[8 * v8 + 3]) * inv_l);
                    o.z = pack2<kBf16>(__uint_as_float(r[8 * v8 + 4]) * inv_l, __uint_as_float(r[8 * v8 + 5]) * inv_l);
                    o.w = pack2<kBf16>(__uint_as_float(r[8 * v8 + 6]) * inv_l, __uint_as_float(r[8 * v8 + 7]) * inv_l);
                    if (s_row < p.S) reinterpret_cast<uint4 *>(o_row + c * 32)[v8] = o;
                }
            }
            if (s_row < p.S) p.lse[q_row] = (m_used + log2f(l)) * kFwdLn2;
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, kTmemCols);
}

#ifdef LT_FWD_TRACE
extern "C" int lt_dbg_fwd_trace(unsigned long long *out, int reset) {
    if (out && cudaMemcpyFromSymbol(out, g_fwd_trace, sizeof(g_fwd_trace)) != cudaSuccess) return LT_ERR_CUDA;
    if (reset) {
        static unsigned long long zeros[32];
        if (cudaMemcpyToSymbol(g_fwd_trace, zeros, sizeof(zeros)) != cudaSuccess) return LT_ERR_CUDA;
    }
    return LT_OK;
}
#endif

template <int D, bool kBf16>
static int launch_fwd(const lt_half *Q, const lt_half *K, const lt_half *V, lt_half *O, float *LSE,
                      const lt_attn_layout &lay, int B, int Hq, int Hkv, int S, int causal, float scale,
                      void *workspace, cudaStream_t stream) {
    CUtensorMap mq, mk, mv;
    int rc;
    if ((rc = make_bhsd_map(&mq, Q, B, Hq, S, D, lay.q, 128, kBf16)) != LT_OK) return rc;
    if ((rc = make_bhsd_map(&mk, K, B, Hkv, S, D, lay.k, 128, kBf16)) != LT_OK) return rc;
    if ((rc = make_bhsd_map(&mv, V, B, Hkv, S, D, lay.v, 128, kBf16)) != LT_OK) return rc;
    cudaError_t e = cudaMemsetAsync(workspace, 0, kStatusBytes, stream);
    if (e != cudaSuccess) return record_cuda_error("cudaMemsetAsync(status)", e);
    FwdParams prm;
    prm.O = reinterpret_cast<__half *>(O);
    prm.lse = LSE;
    prm.o_st = lay.o;
    prm.status = reinterpret_cast<unsigned int *>(workspace);
    prm.B = B; prm.Hq = Hq; prm.Hkv = Hkv; prm.S = S; prm.causal = causal ? 1 : 0;
    prm.scale = scale;
    // at least 120 KB, so that one CTA (which takes all 512 tensor-memory columns) lives on an SM
    const size_t smem = std::max<size_t>(sizeof(FwdSmem<D>) + 1024, 120 * 1024);
    e = cudaFuncSetAttribute(fwd_kernel<D, kBf16>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return record_cuda_error("cudaFuncSetAttribute(fwd)", e);
    const int n_tiles = (S + kFwdTileRows - 1) / kFwdTileRows;
    const int grid = B * Hq * ((n_tiles + 1) / 2);
    fwd_kernel<D, kBf16><<<grid, kFwdThreads, smem, stream>>>(mq, mk, mv, prm);
    e = cudaGetLastError();
    if (e != cudaSuccess) return record_cuda_error("fwd_kernel launch", e);
    return LT_OK;
}

// Internal streams and events of the host-buffer entry point, created on first use per device.
constexpr int kHostMaxChunks = 8, kHostMaxDevices = 64;
struct HostPipe {
    bool ready = false;
    cudaStream_t s_in = nullptr, s_out = nullptr;
    cudaEvent_t ev_start = nullptr, ev_out = nullptr, ev_in[kHostMaxChunks] = {}, ev_comp[kHostMaxChunks] = {};
};
static HostPipe g_host_pipe[kHostMaxDevices];
static std::mutex g_host_pipe_mu;

}  // namespace lt

extern "C" {

size_t lt_attn_fwd_workspace_bytes(int B, int Hq, int Hkv, int S, int D) {
    if (lt::check_shape(B, Hq, Hkv, S, D, 1.0f) != LT_OK) return 0;
    return lt::kStatusBytes;
}

int lt_attn_fwd_num_launches(void) { return 1; }

int lt_attn_fwd(const lt_half *Q, const lt_half *K, const lt_half *V, lt_half *O, float *LSE, int B, int Hq, int Hkv,
                int S, int D, int causal, float scale, void *workspace, size_t workspace_bytes, lt_stream_t stream) {
    return lt_attn_fwd_strided(Q, K, V, O, LSE, nullptr, B, Hq, Hkv, S, D, causal, scale, workspace, workspace_bytes,
                               stream);
}

static int fwd_entry(const lt_half *Q, const lt_half *K, const lt_half *V, lt_half *O, float *LSE,
                     const lt_attn_layout *layout, int B, int Hq, int Hkv, int S, int D, int causal, float scale,
                     void *workspace, size_t workspace_bytes, lt_stream_t stream, bool bf16) {
    using namespace lt;
    if (!Q || !K || !V || !O || !LSE) return LT_ERR_INVALID_ARG;
    int rc = check_shape(B, Hq, Hkv, S, D, scale);
    if (rc != LT_OK) return rc;
    lt_attn_layout lay = contiguous_layout(Hq, Hkv, S, D);
    if (layout) {
        // the forward reads q, k, v, o only; the other entries may be left unset
        lay.q = layout->q; lay.k = layout->k; lay.v = layout->v; lay.o = layout->o;
        if ((rc = check_layout(lay, D)) != LT_OK) return rc;
    }
    const void *ptrs[] = {Q, K, V, O};
    for (const void *ptr : ptrs)
        if (!aligned16(ptr)) return LT_ERR_UNSUPPORTED;
    if ((reinterpret_cast<uintptr_t>(LSE) & 3u) != 0) return LT_ERR_UNSUPPORTED;  // fp32, read and written one at a time
    if (!workspace || !aligned256(workspace) || workspace_bytes < lt_attn_fwd_workspace_bytes(B, Hq, Hkv, S, D))
        return LT_ERR_WORKSPACE;
    if ((rc = check_device()) != LT_OK) return rc;
    if (bf16) {
        if (D == 64) return launch_fwd<64, true>(Q, K, V, O, LSE, lay, B, Hq, Hkv, S, causal, scale, workspace, stream);
        return launch_fwd<128, true>(Q, K, V, O, LSE, lay, B, Hq, Hkv, S, causal, scale, workspace, stream);
    }
    if (D == 64) return launch_fwd<64, false>(Q, K, V, O, LSE, lay, B, Hq, Hkv, S, causal, scale, workspace, stream);
    return launch_fwd<128, false>(Q, K, V, O, LSE, lay, B, Hq, Hkv, S, causal, scale, workspace, stream);
}

int lt_attn_fwd_strided(const lt_half *Q, const lt_half *K, const lt_half *V, lt_half *O, float *LSE,
                        const lt_attn_layout *layout, int B, int Hq, int Hkv, int S, int D, int causal, float scale,
                        void *workspace, size_t workspace_bytes, lt_stream_t stream) {
    return fwd_entry(Q, K, V, O, LSE, layout, B, Hq, Hkv, S, D, causal, scale, workspace, workspace_bytes, stream,
                     false);
}

int lt_attn_fwd_bf16(const lt_bf16 *Q, const lt_bf16 *K, const lt_bf16 *V, lt_bf16 *O, float *LSE,
                     const lt_attn_layout *layout, int B, int Hq, int Hkv, int S, int D, int causal, float scale,
                     void *workspace, size_t workspace_bytes, lt_stream_t stream) {
    return fwd_entry(Q, K, V, O, LSE, layout, B, Hq, Hkv, S, D, causal, scale, workspace, workspace_bytes, stream,
                     true);
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

    // ---- chunks of (batch, kv head) units: the host-to-device copy of one chunk, the kernels of the
    // previous one and the device-to-host copy of the one before run at the same time (two copy engines
    // and the SMs), on two internal streams beside the caller's.  A chunk is a contiguous slice of every
    // tensor and a problem of its own with B = 1.
    const int G = Hq / Hkv;
    const int n_units = B * Hkv;
    const long long n_tiles = padded_rows(S) / 128;
    const long long unit_iters = static_cast<long long>(G) * (causal ? n_tiles * (n_tiles + 1) / 2 : n_tiles * n_tiles);
    // Few, large chunks (a copy of a few MB carries tens of microseconds of fixed cost, and a chunk's kernels take
    // 0.2 ms however small it is); the last chunk is the smallest, because its kernels and its copy back are what is
    // left to do when the input copy ends.
    int bounds[kHostMaxChunks + 1];
    int n_chunks = 1;
    bounds[0] = 0;
    bounds[1] = n_units;
    if (unit_iters * n_units >= 3000 && n_units > 1) {  // otherwise not worth the extra streams
        const int percent[4] = {30, 60, 85, 100};  // cumulative shares of the four chunks
        n_chunks = 0;
        for (int c = 0; c < 4; ++c) {
            int end = c == 3 ? n_units : (n_units * percent[c] + 50) / 100;
            if (end <= bounds[n_chunks]) continue;  // fewer units than chunks
            bounds[++n_chunks] = end;
        }
    }

    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return record_cuda_error("cudaGetDevice", e);
    if (dev < 0 || dev >= kHostMaxDevices) n_chunks = 1;
    std::lock_guard<std::mutex> lock(g_host_pipe_mu);
    HostPipe *pipe = nullptr;
    if (n_chunks > 1) {
        pipe = &g_host_pipe[dev];
        if (!pipe->ready) {
            bool ok = cudaStreamCreateWithFlags(&pipe->s_in, cudaStreamNonBlocking) == cudaSuccess &&
                      cudaStreamCreateWithFlags(&pipe->s_out, cudaStreamNonBlocking) == cudaSuccess &&
                      cudaEventCreateWithFlags(&pipe->ev_start, cudaEventDisableTiming) == cudaSuccess &&
                      cudaEventCreateWithFlags(&pipe->ev_out, cudaEventDisableTiming) == cudaSuccess;
            for (int c = 0; c < kHostMaxChunks && ok; ++c)
                ok = cudaEventCreateWithFlags(&pipe->ev_in[c], cudaEventDisableTiming) == cudaSuccess &&
                     cudaEventCreateWithFlags(&pipe->ev_comp[c], cudaEventDisableTiming) == cudaSuccess;
            if (!ok) return record_cuda_error("stream/event creation for the host pipeline", cudaGetLastError());
            pipe->ready = true;
        }
    }
    cudaStream_t s_in = pipe ? pipe->s_in : stream, s_out = pipe ? pipe->s_out : stream;
#define LT_CUDA(call, what)                      \
    if ((e = (call)) != cudaSuccess) return record_cuda_error(what, e)
    if (pipe) {
        // nothing of this call may start before the work already queued on the caller's stream
        LT_CUDA(cudaEventRecord(pipe->ev_start, stream), "cudaEventRecord");
        LT_CUDA(cudaStreamWaitEvent(s_in, pipe->ev_start, 0), "cudaStreamWaitEvent");
        LT_CUDA(cudaStreamWaitEvent(s_out, pipe->ev_start, 0), "cudaStreamWaitEvent");
    }
    for (int c = 0; c < n_chunks; ++c) {
        const int u0 = bounds[c], u1 = bounds[c + 1];
        const int hkv = u1 - u0, hq = hkv * G;
        const size_t oq = static_cast<size_t>(u0) * G * S * D, ok_ = static_cast<size_t>(u0) * S * D;  // elements
        const size_t ol = static_cast<size_t>(u0) * G * S;
        const size_t cq = static_cast<size_t>(hq) * S * D * 2, ck = static_cast<size_t>(hkv) * S * D * 2;
        const size_t cl = static_cast<size_t>(hq) * S * 4;
        LT_CUDA(cudaMemcpyAsync(d_Q + oq, Q + oq, cq, cudaMemcpyHostToDevice, s_in), "cudaMemcpyAsync");
        LT_CUDA(cudaMemcpyAsync(d_K + ok_, K + ok_, ck, cudaMemcpyHostToDevice, s_in), "cudaMemcpyAsync");
        LT_CUDA(cudaMemcpyAsync(d_V + ok_, V + ok_, ck, cudaMemcpyHostToDevice, s_in), "cudaMemcpyAsync");
        LT_CUDA(cudaMemcpyAsync(d_dO + oq, dO + oq, cq, cudaMemcpyHostToDevice, s_in), "cudaMemcpyAsync");
        if (pipe) {
            LT_CUDA(cudaEventRecord(pipe->ev_in[c], s_in), "cudaEventRecord");
            LT_CUDA(cudaStreamWaitEvent(stream, pipe->ev_in[c], 0), "cudaStreamWaitEvent");
        }
        rc = lt_attn_fwd(d_Q + oq, d_K + ok_, d_V + ok_, d_O + oq, d_lse + ol, 1, hq, hkv, S, D, causal, scale, fwd_ws,
                         kStatusBytes, stream);
        if (rc != LT_OK) return rc;
        rc = lt_attn_bwd(d_Q + oq, d_K + ok_, d_V + ok_, d_O + oq, d_dO + oq, d_lse + ol, d_dQ + oq, d_dK + ok_,
                         d_dV + ok_, 1, hq, hkv, S, D, causal, scale, ws, ws_bytes, stream);
        if (rc != LT_OK) return rc;
        if (pipe) {
            LT_CUDA(cudaEventRecord(pipe->ev_comp[c], stream), "cudaEventRecord");
            LT_CUDA(cudaStreamWaitEvent(s_out, pipe->ev_comp[c], 0), "cudaStreamWaitEvent");
        }
        if (O) LT_CUDA(cudaMemcpyAsync(O + oq, d_O + oq, cq, cudaMemcpyDeviceToHost, s_out), "cudaMemcpyAsync");
        if (LSE) LT_CUDA(cudaMemcpyAsync(LSE + ol, d_lse + ol, cl, cudaMemcpyDeviceToHost, s_out), "cudaMemcpyAsync");
        LT_CUDA(cudaMemcpyAsync(dQ + oq, d_dQ + oq, cq, cudaMemcpyDeviceToHost, s_out), "cudaMemcpyAsync");
        LT_CUDA(cudaMemcpyAsync(dK + ok_, d_dK + ok_, ck, cudaMemcpyDeviceToHost, s_out), "cudaMemcpyAsync");
        LT_CUDA(cudaMemcpyAsync(dV + ok_, d_dV + ok_, ck, cudaMemcpyDeviceToHost, s_out), "cudaMemcpyAsync");
    }
    if (pipe) {
        // the caller's stream is done when the last copy back is
        LT_CUDA(cudaEventRecord(pipe->ev_out, s_out), "cudaEventRecord");
        LT_CUDA(cudaStreamWaitEvent(stream, pipe->ev_out, 0), "cudaStreamWaitEvent");
    }
#undef LT_CUDA
    return LT_OK;
}

}  // extern "C"
