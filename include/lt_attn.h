/*
 * lt_attn.h -- C ABI of the B200 (sm_100a) FP16 attention forward / backward library.
 *
 * The operation is the Attention Backward of a dense decoder layer as the paper's
 * execution backend states it (Section 4.1, "Memory-resident Attention Backward",
 * Algorithm 1):  GP = GO V^T,  GS = SoftmaxBackward(P, GP),  GV = P^T GO,
 * GQ = GS K,  GK = GS^T Q, with the probability tile P as forward state.  By default P is
 * not stored by the forward: lt_attn_bwd rebuilds it tile by tile from the row log-sum-exp.
 * lt_attn_save_p and lt_attn_bwd_saved_p are the stored-P route of the paper, for comparison.
 *
 * Conventions shared by every entry point
 *   - Tensors are contiguous [B, H, S, D] with D innermost (strided views: the *_strided and
 *     *_bf16 entry points).  Q, O, dO, dQ have H = Hq; K, V, dK, dV have H = Hkv.  LSE is fp32
 *     [B, Hq, S].  fp16 is IEEE binary16.
 *   - Grouped-query attention: query head h reads key/value head h / (Hq / Hkv);
 *     dK and dV are summed over the Hq / Hkv query heads of a group.
 *   - scores = scale * Q K^T with a finite, non-zero scale; causal != 0 hides key j from query i when j > i.
 *     LSE_i = ln sum_j exp(scores_ij) over visible keys (natural logarithm).
 *   - Supported shapes: D in {64, 128}, any S >= 1 (a last tile of fewer than 128 rows is
 *     handled inside the kernels; workspace arrays are sized for S rounded up to 128), Hq % Hkv == 0.
 *     Anything else returns LT_ERR_UNSUPPORTED and launches nothing.
 *   - Unless a function says otherwise pointers are DEVICE pointers, 16-byte aligned (LSE: 4-byte),
 *     owned by the caller, and must stay valid until the stream reaches the end of the
 *     call's work.  Inputs are never written.  Outputs are fully overwritten.
 *   - Calls only enqueue work on `stream` and return; they do not synchronise and
 *     allocate no device memory.  Two calls may overlap on the GPU only if they use
 *     different workspaces.
 *   - Value range of the backward: dS is rounded to fp16 (bf16) after multiplication by a power of two
 *     picked per call from max ||dO_row||, max |delta| and max ||V_row|| (their product bounds |dS|), so
 *     gradients keep their relative accuracy for upstream gradients and values of any usual magnitude.
 *     Non-finite inputs make that bound infinite; the most cautious factor is then used.
 *   - Return value: LT_OK or an lt_status error.  Errors found on the host launch
 *     nothing.  A device-side wait that gave up (a bounded spin on a barrier ran out)
 *     is recorded in the workspace and read back with lt_attn_check_status.
 *   - The library targets the current CUDA device, which must be compute capability 10.x.
 */
#ifndef LT_ATTN_H_
#define LT_ATTN_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum lt_status {
    LT_OK = 0,
    LT_ERR_INVALID_ARG = 1,    /* NULL pointer, non-positive size, Hq % Hkv != 0, zero or non-finite scale */
    LT_ERR_UNSUPPORTED = 2,    /* shape, alignment or device outside the supported set */
    LT_ERR_WORKSPACE = 3,      /* workspace NULL, misaligned (256 B) or too small */
    LT_ERR_CUDA = 4,           /* a CUDA runtime/driver call failed; see lt_last_cuda_error */
    LT_ERR_DEVICE_TIMEOUT = 5  /* a bounded device-side wait expired (lt_attn_check_status only) */
} lt_status;

/* ABI-compatible with cudaStream_t. */
typedef struct CUstream_st *lt_stream_t;
/* ABI-compatible with cudaEvent_t. */
typedef struct CUevent_st *lt_event_t;
/* fp16 storage type (bit pattern of an IEEE binary16). */
typedef unsigned short lt_half;
/* bfloat16 storage (the upper 16 bits of an IEEE binary32) */
typedef unsigned short lt_bf16;

/* Bytes of caller-owned device workspace the calls below need; 0 means the shape is
 * not supported.  The workspace must be 256-byte aligned.  Layout (backward), with S_pad = S
 * rounded up to a multiple of 128: a 256-byte status block (word 0: code of a wait that gave up;
 * words 1, 2, 4: the three maxima above as fp32 bits; word 3: work-item counter), -delta and -LSE/scale as 16-byte rows
 * of fp16 (hi, lo, 0 x 6) with 256*hi + lo = value, [B,Hq,S_pad] rows each, an fp32 dQ accumulator
 * [B,Hq,S_pad,D], and, for the grouped-query shapes whose groups are split over work items (see
 * lt_attn_bwd_num_launches), fp32 dK and dV sums [B,Hkv,S_pad,D] each. */
size_t lt_attn_fwd_workspace_bytes(int B, int Hq, int Hkv, int S, int D);
size_t lt_attn_bwd_workspace_bytes(int B, int Hq, int Hkv, int S, int D);

/* Forward: O = softmax(scale Q K^T [+ causal mask]) V, and the row log-sum-exp.
 * The forward step that produces the state Algorithm 1 requires (the paper saves P;
 * this library saves LSE, from which the backward recomputes P).
 *   in : Q [B,Hq,S,D], K, V [B,Hkv,S,D]  fp16
 *   out: O [B,Hq,S,D] fp16, LSE [B,Hq,S] fp32 */
int lt_attn_fwd(const lt_half *Q, const lt_half *K, const lt_half *V,
                lt_half *O, float *LSE,
                int B, int Hq, int Hkv, int S, int D, int causal, float scale,
                void *workspace, size_t workspace_bytes, lt_stream_t stream);

/* Backward (Algorithm 1): dQ, dK, dV of L with dO = dL/dO.
 *   delta = rowsum(dO * O)                          preprocess kernel
 *   P     = exp(scale Q K^T - LSE)  (masked)        recomputed per tile
 *   dV   += P^T dO;  dP = dO V^T;  dS = P * (dP - delta)
 *   dQ   += scale dS K;  dK += scale dS^T Q
 *   in : Q, O, dO [B,Hq,S,D] fp16; K, V [B,Hkv,S,D] fp16; LSE [B,Hq,S] fp32
 *   out: dQ [B,Hq,S,D], dK, dV [B,Hkv,S,D] fp16 (overwritten, not accumulated into)
 * dQ is accumulated in fp32 in the workspace with atomic adds, so its last bits may
 * differ between runs; dK and dV are bitwise reproducible, except on the grouped-query shapes
 * whose groups are split over work items (see lt_attn_bwd_num_launches), where they are summed
 * the same way.  The main and conversion kernels are launched with programmatic stream
 * serialisation (each starts under the tail of its predecessor and waits inside for it). */
int lt_attn_bwd(const lt_half *Q, const lt_half *K, const lt_half *V,
                const lt_half *O, const lt_half *dO, const float *LSE,
                lt_half *dQ, lt_half *dK, lt_half *dV,
                int B, int Hq, int Hkv, int S, int D, int causal, float scale,
                void *workspace, size_t workspace_bytes, lt_stream_t stream);

/* lt_attn_bwd with two optional CUDA events recorded on `stream` immediately before and
 * after the main (tensor-core) kernel, so a benchmark can time that kernel inside a
 * normal call.  Either event may be NULL.  Everything else is as for lt_attn_bwd. */
int lt_attn_bwd_profiled(const lt_half *Q, const lt_half *K, const lt_half *V,
                         const lt_half *O, const lt_half *dO, const float *LSE,
                         lt_half *dQ, lt_half *dK, lt_half *dV,
                         int B, int Hq, int Hkv, int S, int D, int causal, float scale,
                         void *workspace, size_t workspace_bytes, lt_stream_t stream,
                         lt_event_t main_begin, lt_event_t main_end);

/* lt_attn_bwd for callers that cannot allocate device memory (the paper has no counterpart
 * to this entry point).  Some hosts of this library may not call cudaMalloc at the point
 * where they need the backward: code running inside a memory pool that must not grow, a
 * plugin that is handed tensors but no allocator, a step that has to stay allocation-free
 * after start-up.  For them the scratch that lt_attn_bwd takes as `workspace` comes from a
 * fixed array of LT_ATTN_BWD_NOALLOC_MAX_SCRATCH_BYTES inside the library itself, which every
 * GPU that loads the library holds until the process ends.  Inputs and outputs are still the
 * caller's device tensors, with the meaning and layout of lt_attn_bwd.
 *   - Shapes whose lt_attn_bwd_workspace_bytes() exceeds the built-in scratch (roughly
 *     B*Hq*S*D above four million elements) return LT_ERR_WORKSPACE; lt_last_cuda_error()
 *     then names both sizes.  Nothing is launched in that case.
 *   - The call allocates nothing: no cudaMalloc/cudaFree and no allocating library routine.
 *   - The first call on each device looks up the array's device address (one runtime query,
 *     under a lock); make that first call before any CUDA stream capture begins.
 *   - All calls on a device share the one scratch array.  Each call clears what it needs at
 *     zero itself, so an earlier call's leftovers are harmless, but two calls that overlap
 *     on the GPU (different streams) race on it: serialise them.
 *   - The caller has no pointer to the scratch, so a device-side wait that gave up is read back
 *     with lt_attn_bwd_noalloc_check_status(stream): it synchronises `stream`, copies the status word
 *     of the current device's scratch to the host (4 bytes; nothing is allocated and no pointer is
 *     handed out) and returns what lt_attn_check_status would. */
#define LT_ATTN_BWD_NOALLOC_MAX_SCRATCH_BYTES (18u * 1024u * 1024u)
int lt_attn_bwd_noalloc(const lt_half *Q, const lt_half *K, const lt_half *V,
                        const lt_half *O, const lt_half *dO, const float *LSE,
                        lt_half *dQ, lt_half *dK, lt_half *dV,
                        int B, int Hq, int Hkv, int S, int D, int causal, float scale,
                        lt_stream_t stream);
int lt_attn_bwd_noalloc_check_status(lt_stream_t stream);

/* Layouts other than contiguous [B,H,S,D].  Each tensor is described by the element strides of
 * its batch, head and row (sequence position) indices; the D elements of a row are always
 * contiguous.  Element (b, h, s, d) lives at base + b*batch + h*head + s*row + d.  A fused
 * QKV projection output [B, S, (Hq + 2 Hkv) * D], or a [B,S,H,D] tensor, is such a view.
 * Every stride must be a positive multiple of 8 elements (16 bytes) and row >= D; views must not
 * overlap themselves.  LSE is always contiguous [B,Hq,S].  The paper fixes no memory layout. */
typedef struct lt_tensor_strides {
    long long batch, head, row;
} lt_tensor_strides;
typedef struct lt_attn_layout {
    lt_tensor_strides q, k, v, o, d_o, dq, dk, dv;  /* the forward reads q, k, v, o only */
} lt_attn_layout;

/* lt_attn_fwd / lt_attn_bwd on strided views.  `layout` is a HOST pointer read during the call
 * (NULL means contiguous [B,H,S,D], i.e. exactly lt_attn_fwd / lt_attn_bwd).  Same workspace
 * sizes, status codes and error behaviour; a stride that breaks the rules above returns
 * LT_ERR_UNSUPPORTED and launches nothing. */
int lt_attn_fwd_strided(const lt_half *Q, const lt_half *K, const lt_half *V,
                        lt_half *O, float *LSE, const lt_attn_layout *layout,
                        int B, int Hq, int Hkv, int S, int D, int causal, float scale,
                        void *workspace, size_t workspace_bytes, lt_stream_t stream);
int lt_attn_bwd_strided(const lt_half *Q, const lt_half *K, const lt_half *V,
                        const lt_half *O, const lt_half *dO, const float *LSE,
                        lt_half *dQ, lt_half *dK, lt_half *dV, const lt_attn_layout *layout,
                        int B, int Hq, int Hkv, int S, int D, int causal, float scale,
                        void *workspace, size_t workspace_bytes, lt_stream_t stream);

/* The same two computations with every 16-bit tensor (Q, K, V, O, dO, dQ, dK, dV) in bfloat16
 * instead of fp16; LSE stays fp32.  Products run on the same tensor-core path with bf16 operands
 * and fp32 accumulation; P and dS are rounded to bf16 (8 significant bits) before their products, so
 * the gradients carry about 2^-9 relative rounding per element where the fp16 path carries 2^-11.
 * `layout` as for the strided entry points (NULL = contiguous [B,H,S,D]).  Workspace sizes, status
 * codes and error behaviour are those of lt_attn_fwd / lt_attn_bwd.  The paper's datapath is FP16
 * (Section 4.1); bf16 is the format most current training stacks hand to the same operator. */
int lt_attn_fwd_bf16(const lt_bf16 *Q, const lt_bf16 *K, const lt_bf16 *V,
                     lt_bf16 *O, float *LSE, const lt_attn_layout *layout,
                     int B, int Hq, int Hkv, int S, int D, int causal, float scale,
                     void *workspace, size_t workspace_bytes, lt_stream_t stream);
int lt_attn_bwd_bf16(const lt_bf16 *Q, const lt_bf16 *K, const lt_bf16 *V,
                     const lt_bf16 *O, const lt_bf16 *dO, const float *LSE,
                     lt_bf16 *dQ, lt_bf16 *dK, lt_bf16 *dV, const lt_attn_layout *layout,
                     int B, int Hq, int Hkv, int S, int D, int causal, float scale,
                     void *workspace, size_t workspace_bytes, lt_stream_t stream);

/* Attention Backward with the forward pass's saved probabilities (Section 4.1: the paper's backward
 * loads the probability tile P_ij the forward saved, where lt_attn_bwd recomputes it from LSE).
 *
 * lt_attn_save_p writes that forward state from Q, K and the forward's LSE: P = exp(scale*Q K^T - LSE)
 * rounded to fp16, stored as transposed tiles.  Tile (b, h, j, i) - key tile j, query tile i of query
 * head h, tiles of 128 rows, nT = ceil(S/128) - is a 32 KB block at tile index ((b*Hq + h)*nT + j)*nT + i
 * of `P`; inside it, element (key, query) sits at fp16 offset (query/8)*1024 + key*8 + query%8 (sixteen
 * blocks of eight query columns, each [128 keys][8 queries], so that a warp holding consecutive key
 * rows moves 512 contiguous bytes per access).  `P` holds lt_attn_p_store_bytes() bytes
 * (B*Hq*nT*nT*32768; 0 for an unsupported shape) and is 256-byte aligned.  Entries hidden by the
 * causal mask or past the end of the sequence are zero; with causal != 0, tiles with i < j are not
 * written and never read.  Q, K, LSE as for lt_attn_bwd (contiguous [B,H,S,D], fp16); `workspace` needs
 * only the 256-byte status block.  One kernel launch.  lt_attn_save_p stands in for a forward pass that would
 * write P as it goes (it recomputes the scores from Q, K and LSE); it is there to produce the paper's forward
 * state for lt_attn_bwd_saved_p, not tuned, and runs at about a third of the HBM write rate of its output.
 *
 * lt_attn_bwd_saved_p computes dQ, dK, dV as lt_attn_bwd does, with `P` (the store above, same shape
 * arguments and mask) in place of LSE: the main kernel issues no S = Q K^T product and no exponentials;
 * it reads each tile of P once (32 KB per tile pair, B*Hq*nT*(nT+1)/2 tile pairs under a causal mask).
 * Contiguous fp16 tensors only; workspace of lt_attn_bwd_workspace_bytes() bytes; three launches; status
 * and error behaviour as lt_attn_bwd.  P carries fp16 rounding (and flushes probabilities below 2^-24
 * to zero), which the recompute path does not, so its gradients are slightly less accurate. */
size_t lt_attn_p_store_bytes(int B, int Hq, int Hkv, int S, int D);
int lt_attn_save_p(const lt_half *Q, const lt_half *K, const float *LSE, lt_half *P,
                   int B, int Hq, int Hkv, int S, int D, int causal, float scale,
                   void *workspace, size_t workspace_bytes, lt_stream_t stream);
int lt_attn_bwd_saved_p(const lt_half *Q, const lt_half *K, const lt_half *V,
                        const lt_half *O, const lt_half *dO, const lt_half *P,
                        lt_half *dQ, lt_half *dK, lt_half *dV,
                        int B, int Hq, int Hkv, int S, int D, int causal, float scale,
                        void *workspace, size_t workspace_bytes, lt_stream_t stream);

/* FP16 GEMM, the linear-layer primitive of the paper's backend (Section 4.1, "FP16 GEMM assembly
 * pipeline"; its profiled shapes are in Section 6.6):  C[M,N] = A[M,K] W[N,K]^T.
 *   in : A [M,K] fp16 row-major (activations), W [N,K] fp16 row-major (a linear layer's weight as stored)
 *   out: C [M,N] fp16 row-major, fully overwritten; products accumulate in fp32
 * Any M, N >= 1; K >= 8 and a multiple of 8 (16-byte row pitch for the tile loads); otherwise
 * LT_ERR_UNSUPPORTED.  Device pointers, 16-byte aligned, owned by the caller.  `workspace` holds only
 * the 256-byte status block (lt_gemm_f16_workspace_bytes()); read it with lt_attn_check_status.
 * Enqueues one kernel on `stream`; allocates nothing; does not synchronise.  With more than 128 rows in A the
 * kernel runs as clusters of two CTAs that share 256x256 output tiles (pair products); LT_GEMM_SINGLE_CTA=1 in the
 * environment, read at the first call, keeps the single-CTA kernel. */
size_t lt_gemm_f16_workspace_bytes(void);
int lt_gemm_f16(const lt_half *A, const lt_half *W, lt_half *C, int M, int N, int K,
                void *workspace, size_t workspace_bytes, lt_stream_t stream);
/* The same product with bfloat16 A, W and C (fp32 accumulation); everything else as lt_gemm_f16. */
int lt_gemm_bf16(const lt_bf16 *A, const lt_bf16 *W, lt_bf16 *C, int M, int N, int K,
                 void *workspace, size_t workspace_bytes, lt_stream_t stream);

/* Same computation as lt_attn_fwd followed by lt_attn_bwd, but every tensor pointer is
 * a HOST pointer (pinned memory makes the copies asynchronous).  `arena` is a caller-
 * owned DEVICE buffer of at least lt_attn_host_arena_bytes() bytes, 256-byte aligned,
 * that holds the device copies and the workspace.  The call enqueues the host-to-device
 * copies of Q, K, V, dO, the two kernels' work and the device-to-host copies of
 * O, LSE, dQ, dK, dV on `stream`; the host outputs are valid once the stream is
 * synchronised.  O and LSE may be NULL if the caller does not want them back.
 * Large problems are cut into chunks of (batch, kv head) units so that the copy in of one chunk, the
 * kernels of the previous one and the copy back of the one before overlap; the copies run on two
 * streams the library creates once per device (no device memory is allocated), forked from and
 * joined back into `stream` with events, so the ordering guarantees above are unchanged.  The status
 * blocks inside the arena are those of the last chunk. */
size_t lt_attn_host_arena_bytes(int B, int Hq, int Hkv, int S, int D);
int lt_attn_fwd_bwd_host(const lt_half *Q, const lt_half *K, const lt_half *V, const lt_half *dO,
                         lt_half *O, float *LSE, lt_half *dQ, lt_half *dK, lt_half *dV,
                         int B, int Hq, int Hkv, int S, int D, int causal, float scale,
                         void *arena, size_t arena_bytes, lt_stream_t stream);

/* Synchronises `stream`, reads the status block of `workspace` and returns LT_OK,
 * LT_ERR_DEVICE_TIMEOUT (a kernel abandoned a wait; outputs are invalid) or LT_ERR_CUDA. */
int lt_attn_check_status(const void *workspace, lt_stream_t stream);

/* Static strings; never NULL. */
const char *lt_status_string(int status);
const char *lt_last_cuda_error(void);

/* Number of kernels one call enqueues for this shape (for launch accounting by benchmarks): the
 * backward's preprocess, main and dQ-conversion kernels, plus the dK/dV conversion on grouped-query shapes
 * with fewer than about 1.5 key-tile work items per multiprocessor, where a group's query heads are split
 * over several items (4 instead of 3); 0 for an unsupported shape.  The forward enqueues one kernel. */
int lt_attn_bwd_num_launches(int B, int Hq, int Hkv, int S, int D, int causal);
int lt_attn_fwd_num_launches(void);

#ifdef __cplusplus
}
#endif
#endif /* LT_ATTN_H_ */
