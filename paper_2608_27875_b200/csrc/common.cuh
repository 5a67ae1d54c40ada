// Shared host/device helpers of the hyq library (no method arithmetic here).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/hyq.h"

#define HYQ_D 128
#define HYQ_BLOCK_TOKENS 64

namespace hyq {

__device__ __forceinline__ float bf16_bits_to_f32(uint32_t h) { return __uint_as_float(h << 16); }

// low / high bf16 of a packed 32-bit word
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

static inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
__host__ __device__ constexpr size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

static inline int launch_status() { return cudaGetLastError() == cudaSuccess ? HYQ_OK : HYQ_ERR_CUDA; }

// internal launchers (defined in the kernel files)
int launch_quantize(const void* x, long n_heads, int L, int block_tokens, int format, void* codes, float* scales, cudaStream_t st);
static inline bool block_tokens_ok(int bt) { return bt == 32 || bt == 64 || bt == 128; }
int launch_select(const void* q, const void* k, int B, int Hq, int Hkv, int Lq, int Lk, int window, int n_tail,
                  int k_sel, int32_t* idx_out, void* ws, cudaStream_t st);
size_t select_workspace_bytes(int B, int Hq, int Lk, int window);
int launch_topk(const double* scores, long rows, int P, int k_sel, int32_t* idx_out, cudaStream_t st);
size_t select_mass_workspace_bytes(int B, int Hq, int Lk, int window, int n_queries);
int launch_select_mass(const void* q, const void* k, int B, int Hq, int Hkv, int Lq, int Lk, int window, int n_queries,
                       int k_sel, double alpha, int32_t* idx_out, void* ws, cudaStream_t st);
int launch_select_static(const void* q, const void* k, int B, int Hq, int Hkv, int Lq, int Lk, int window, int n_tail,
                         int k_sel, int32_t* idx_out, cudaStream_t st);

}  // namespace hyq
