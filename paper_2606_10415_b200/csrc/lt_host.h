// Host-side helpers shared by the entry points: argument checks, the TMA tensor-map
// encoder (fetched from the driver at run time so the library links without libcuda),
// and the last-error string.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/lt_attn.h"

namespace lt {

void set_last_error(const char *what, const char *detail);
int record_cuda_error(const char *what, cudaError_t err);

// LT_OK, or the reason the current device cannot run the kernels.
int check_device();

// Validates the common (B, Hq, Hkv, S, D, scale) arguments.
int check_shape(int B, int Hq, int Hkv, int S, int D, float scale);

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline bool aligned256(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 255u) == 0; }
inline size_t round256(size_t n) { return (n + 255u) & ~static_cast<size_t>(255u); }

// fp16 matrix [rows, cols] row-major viewed as a 2-D tensor; tiles of box_rows x 64
// columns are fetched with the 128-byte swizzle.  Returns LT_OK or LT_ERR_CUDA.
int make_tile_map(CUtensorMap *map, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows);
// 4-D view [batch][head][row][element] of an fp16 (or bf16) tensor with the given element strides (boxes of
// 64 elements x box_rows rows of one head, 128-byte swizzle, zero fill past the last row).
int make_bhsd_map(CUtensorMap *map, const void *base, uint64_t B, uint64_t H, uint64_t S, uint64_t D,
                  const lt_tensor_strides &st, uint32_t box_rows, bool bf16 = false);
// fp32 matrix [rows, cols] row-major (cols a multiple of 32) viewed as a 2-D tensor; tiles of box_rows x 32
// columns (128 bytes per row) with the 128-byte swizzle, for tiled reductions from shared memory.
int make_f32_tile_map(CUtensorMap *map, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows);
// strides of a contiguous [B,H,S,D] tensor
inline lt_tensor_strides contiguous_strides(int H, int S, int D) {
    lt_tensor_strides st;
    st.row = D;
    st.head = static_cast<long long>(S) * D;
    st.batch = static_cast<long long>(H) * S * D;
    return st;
}
// every tensor contiguous [B,H,S,D]
lt_attn_layout contiguous_layout(int Hq, int Hkv, int S, int D);
// LT_OK if every stride of the layout is a positive multiple of 8 elements and rows hold D elements
int check_layout(const lt_attn_layout &lay, int D);
// sequence length rounded up to whole 128-row tiles
inline long long padded_rows(int S) { return (static_cast<long long>(S) + 127) / 128 * 128; }

}  // namespace lt
