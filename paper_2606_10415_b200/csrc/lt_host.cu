// Host-side helpers and the small entry points that launch nothing heavy.
#include "lt_host.h"

#include <stdio.h>
#include <string.h>

#include "lt_common.cuh"

namespace lt {

static thread_local char g_last_error[512] = "no error";

void set_last_error(const char *what, const char *detail) {
    snprintf(g_last_error, sizeof(g_last_error), "%s: %s", what, detail ? detail : "");
}

int record_cuda_error(const char *what, cudaError_t err) {
    set_last_error(what, cudaGetErrorString(err));
    return LT_ERR_CUDA;
}

int check_device() {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return record_cuda_error("cudaGetDevice", e);
    int major = 0;
    e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (e != cudaSuccess) return record_cuda_error("cudaDeviceGetAttribute", e);
    if (major != 10) {
        set_last_error("device", "compute capability 10.x (B200) required");
        return LT_ERR_UNSUPPORTED;
    }
    return LT_OK;
}

int check_shape(int B, int Hq, int Hkv, int S, int D, float scale) {
    if (B <= 0 || Hq <= 0 || Hkv <= 0 || S <= 0 || D <= 0) return LT_ERR_INVALID_ARG;
    if (Hq % Hkv != 0) return LT_ERR_INVALID_ARG;
    if (!isfinite(scale) || scale == 0.f) return LT_ERR_INVALID_ARG;
    if (D != 64 && D != 128) return LT_ERR_UNSUPPORTED;
    // padded row indices (every head rounded up to whole 128-row tiles) must fit 32 bits
    if (static_cast<long long>(B) * Hq * padded_rows(S) >= (1LL << 31)) return LT_ERR_UNSUPPORTED;
    return LT_OK;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encoder() {
    static EncodeTiledFn fn = nullptr;
    if (fn) return fn;
    void *p = nullptr;
    cudaDriverEntryPointQueryResult q;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q);
    if (e != cudaSuccess || q != cudaDriverEntryPointSuccess || !p) {
        set_last_error("cudaGetDriverEntryPoint", "cuTensorMapEncodeTiled not available");
        return nullptr;
    }
    fn = reinterpret_cast<EncodeTiledFn>(p);
    return fn;
}

int make_tile_map(CUtensorMap *map, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    EncodeTiledFn enc = get_encoder();
    if (!enc) return LT_ERR_CUDA;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * sizeof(__half)};
    cuuint32_t box[2] = {64u, box_rows};
    cuuint32_t estr[2] = {1u, 1u};
    CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        char buf[64];
        snprintf(buf, sizeof(buf), "CUresult %d", static_cast<int>(r));
        set_last_error("cuTensorMapEncodeTiled", buf);
        return LT_ERR_CUDA;
    }
    return LT_OK;
}

int make_bhsd_map(CUtensorMap *map, const void *base, uint64_t B, uint64_t H, uint64_t S, uint64_t D,
                  const lt_tensor_strides &st, uint32_t box_rows, bool bf16) {
    EncodeTiledFn enc = get_encoder();
    if (!enc) return LT_ERR_CUDA;
    cuuint64_t dims[4] = {D, S, H, B};
    cuuint64_t strides[3] = {static_cast<cuuint64_t>(st.row) * sizeof(__half),
                             static_cast<cuuint64_t>(st.head) * sizeof(__half),
                             static_cast<cuuint64_t>(st.batch) * sizeof(__half)};
    cuuint32_t box[4] = {64u, box_rows, 1u, 1u};
    cuuint32_t estr[4] = {1u, 1u, 1u, 1u};
    CUresult r = enc(map, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 4,
                     const_cast<void *>(base), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        char buf[64];
        snprintf(buf, sizeof(buf), "CUresult %d", static_cast<int>(r));
        set_last_error("cuTensorMapEncodeTiled", buf);
        return LT_ERR_CUDA;
    }
    return LT_OK;
}

int make_f32_tile_map(CUtensorMap *map, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    EncodeTiledFn enc = get_encoder();
    if (!enc) return LT_ERR_CUDA;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * sizeof(float)};
    cuuint32_t box[2] = {32u, box_rows};
    cuuint32_t estr[2] = {1u, 1u};
    CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void *>(base), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        char buf[64];
        snprintf(buf, sizeof(buf), "CUresult %d", static_cast<int>(r));
        set_last_error("cuTensorMapEncodeTiled(f32)", buf);
        return LT_ERR_CUDA;
    }
    return LT_OK;
}

lt_attn_layout contiguous_layout(int Hq, int Hkv, int S, int D) {
    lt_attn_layout lay;
    lay.q = lay.o = lay.d_o = lay.dq = contiguous_strides(Hq, S, D);
    lay.k = lay.v = lay.dk = lay.dv = contiguous_strides(Hkv, S, D);
    return lay;
}

int check_layout(const lt_attn_layout &lay, int D) {
    const lt_tensor_strides *all[] = {&lay.q, &lay.k, &lay.v, &lay.o, &lay.d_o, &lay.dq, &lay.dk, &lay.dv};
    for (const lt_tensor_strides *st : all) {
        const long long v[3] = {st->batch, st->head, st->row};
        for (long long x : v)
            if (x <= 0 || (x % 8) != 0 || x >= (1LL << 38)) return LT_ERR_UNSUPPORTED;
        if (st->row < D) return LT_ERR_UNSUPPORTED;
    }
    return LT_OK;
}

}  // namespace lt

extern "C" {

const char *lt_status_string(int status) {
    switch (status) {
        case LT_OK: return "ok";
        case LT_ERR_INVALID_ARG: return "invalid argument";
        case LT_ERR_UNSUPPORTED: return "unsupported shape, alignment or device";
        case LT_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case LT_ERR_CUDA: return "CUDA call failed";
        case LT_ERR_DEVICE_TIMEOUT: return "a device-side wait gave up";
        default: return "unknown status";
    }
}

const char *lt_last_cuda_error(void) { return lt::g_last_error; }

int lt_attn_check_status(const void *workspace, lt_stream_t stream) {
    if (!workspace) return LT_ERR_WORKSPACE;
    unsigned int word = 0;
    cudaError_t e = cudaMemcpyAsync(&word, workspace, sizeof(word), cudaMemcpyDeviceToHost, stream);
    if (e != cudaSuccess) return lt::record_cuda_error("cudaMemcpyAsync(status)", e);
    e = cudaStreamSynchronize(stream);
    if (e != cudaSuccess) return lt::record_cuda_error("cudaStreamSynchronize", e);
    if (word != 0) {
        char buf[64];
        snprintf(buf, sizeof(buf), "wait code %u", word);
        lt::set_last_error("device timeout", buf);
        return LT_ERR_DEVICE_TIMEOUT;
    }
    return LT_OK;
}

}  // extern "C"
