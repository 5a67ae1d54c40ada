// Pre-pass of the fused attention: lays out in the caller's workspace what the tensor-core kernel
// streams with TMA.  All kernels are simple, coalesced and bound by memory traffic.
//   - vertical-line bitmask per (b, h) over key positions
//   - gathered vertical-line K rows (bf16) and V rows (fp16) per query head, in ascending position
//     order (the physical "reorder" of Algorithm 2 Stage 1, done per query head because under
//     GQA the heads that share a KV head select different keys)
//   - V in fp16 (full-precision class) and dequantized V^ = code * scale in fp16 (low-bit class):
//     the P.V products run as fp16 x fp16 MMAs
//   - INT4 codes widened to one e4m3 byte each (-7..7 are exact in e4m3), so that the score MMA
//     returns fp32 sums that are exact integers
#include <cuda_fp16.h>
#include <cuda_fp8.h>

#include "attn_common.cuh"

namespace hyq {

// two floats -> fp16 pair, saturated to the largest finite fp16: a value row beyond the documented range
// (|V| < 65504) then degrades the result instead of putting an infinity, and with it NaNs, into the output
__device__ __forceinline__ uint32_t f16x2_sat(float a, float b) {
    const __half2 h2 = __floats2half2_rn(fminf(fmaxf(a, -65504.0f), 65504.0f), fminf(fmaxf(b, -65504.0f), 65504.0f));
    return *reinterpret_cast<const uint32_t*>(&h2);
}

__global__ void vl_bitmask_kernel(const int32_t* __restrict__ idx, long n_heads, int k, int L, int mask_words,
                                  uint32_t* __restrict__ bits) {
    const long e = (long)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= n_heads * k) return;
    const long head = e / k;
    const int j = idx[e];
    if (j >= 0 && j < L) atomicOr(&bits[head * mask_words + (j >> 5)], 1u << (j & 31));
}

// one warp per gathered row: lane copies 4 channels
__global__ void gather_vl_kernel(const __nv_bfloat16* __restrict__ kmat, const __nv_bfloat16* __restrict__ vmat,
                                 const int32_t* __restrict__ idx, int Hq, int Hkv, int L, int k, long n_rows,
                                 __nv_bfloat16* __restrict__ kvl, __half* __restrict__ vvl) {
    const long row = ((long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (row >= n_rows) return;
    const long head = row / k;                       // b * Hq + h
    const int b = (int)(head / Hq), h = (int)(head % Hq), g = Hq / Hkv;
    int j = idx[row];
    j = min(max(j, 0), L - 1);
    const long src = (((long)b * Hkv + h / g) * L + j) * HYQ_D + lane * 4;
    const uint2 kw = *reinterpret_cast<const uint2*>(kmat + src);
    const uint2 vw = *reinterpret_cast<const uint2*>(vmat + src);
    *reinterpret_cast<uint2*>(kvl + row * HYQ_D + lane * 4) = kw;
    uint2 o;
    o.x = f16x2_sat(bf16_lo(vw.x), bf16_hi(vw.x));
    o.y = f16x2_sat(bf16_lo(vw.y), bf16_hi(vw.y));
    *reinterpret_cast<uint2*>(vvl + row * HYQ_D + lane * 4) = o;
}

// V (bf16) -> fp16 and V^ = code * scale -> fp16; one thread per 8 channels
template <int V_FMT>
__global__ void v_to_fp16_kernel(const uint4* __restrict__ v, const uint2* __restrict__ v_codes,
                                 const float* __restrict__ v_scales, int L, int nb, int block_tokens, long n_vec,
                                 uint4* __restrict__ v16, uint4* __restrict__ vh16) {
    const long e = (long)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= n_vec) return;
    const long row = e / (HYQ_D / 8);                // global token row over all (b, kv head)
    const long head = row / L;
    const int tok = (int)(row - head * L);
    const float sc = v_scales[head * nb + tok / block_tokens];
    const uint4 w = __ldg(v + e);
    const uint32_t ws[4] = {w.x, w.y, w.z, w.w};
    uint32_t o[4], oh[4];
#pragma unroll
    for (int c = 0; c < 4; ++c) o[c] = f16x2_sat(bf16_lo(ws[c]), bf16_hi(ws[c]));
    const uint2 cw = __ldg(v_codes + e);
    const uint32_t cs[2] = {cw.x, cw.y};
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        const uint32_t two = (cs[c >> 1] >> ((c & 1) * 16)) & 0xFFFFu;
        float f0, f1;
        if (V_FMT == HYQ_FMT_INT8) {
            f0 = (float)(int8_t)(two & 0xFF);
            f1 = (float)(int8_t)(two >> 8);
        } else {
            const __half2_raw hr = __nv_cvt_fp8x2_to_halfraw2((__nv_fp8x2_storage_t)two, __NV_E4M3);
            const float2 ff = __half22float2(__half2(hr));
            f0 = ff.x;
            f1 = ff.y;
        }
        oh[c] = f16x2_sat(f0 * sc, f1 * sc);
    }
    v16[e] = make_uint4(o[0], o[1], o[2], o[3]);
    vh16[e] = make_uint4(oh[0], oh[1], oh[2], oh[3]);
}

// packed INT4 codes -> one e4m3 byte per code; one thread per 8 codes
__global__ void int4_to_e4m3_kernel(const uint32_t* __restrict__ packed, long n_words, uint2* __restrict__ out) {
    const long e = (long)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= n_words) return;
    // e4m3 encodings of 0..8 (1 = 0x38, 2 = 0x40, 3 = 0x44, ...); sign goes to bit 7
    const uint32_t w = __ldg(packed + e);
    uint32_t o[2] = {0u, 0u};
#pragma unroll
    for (int n = 0; n < 8; ++n) {
        const int v = ((int)(w << (28 - 4 * n))) >> 28;
        const int a = abs(v);
        // magnitudes 0..8 -> 0x00,0x38,0x40,0x44,0x48,0x4A,0x4C,0x4E,0x50
        const uint64_t lut = 0x4E4C4A4844403800ull;
        uint32_t code = (a == 8) ? 0x50u : (uint32_t)((lut >> (8 * a)) & 0xFF);
        code |= (v < 0) ? 0x80u : 0u;
        o[n >> 2] |= code << ((n & 3) * 8);
    }
    out[e] = make_uint2(o[0], o[1]);
}

// one thread per vertical-line index: the byte 0xFC (-inf in e5m2) into element 0 of the key's row of its tile's operand
__global__ void vl_mask_tiles_kernel(const int32_t* __restrict__ idx, long n_heads, int k, int L, int tiles_per_head,
                                     uint8_t* __restrict__ tiles) {
    const long e = (long)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= n_heads * k) return;
    const long head = e / k;
    const int j = __ldg(idx + e);
    if (j >= 0 && j < L) tiles[(head * tiles_per_head + (j >> 6)) * VL_TILE_BYTES + (j & 63) * 16] = 0xFC;
}

int launch_vl_bitmask(const int32_t* idx, long n_heads, int k, int L, int mask_words, uint32_t* bits, cudaStream_t st) {
    if (cudaMemsetAsync(bits, 0, (size_t)n_heads * mask_words * 4, st) != cudaSuccess) return HYQ_ERR_CUDA;
    if (k <= 0) return HYQ_OK;
    const long n = n_heads * k;
    vl_bitmask_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(idx, n_heads, k, L, mask_words, bits);
    return launch_status();
}

// ---------------------------------------------------------------------------------------------
int tc_key_splits(const hyq_attn_args& a) {
    const int Lq = query_rows(a);
    if (Lq >= a.L) return 1;                                     // the whole prefill fills the GPU by itself
    const long ctas = (long)((Lq + 255) / 256) * a.Hq * a.B;
    const long target = 2 * 148;                                 // about two CTAs per SM
    if (ctas >= target / 2) return 1;
    const int key_tiles = (a.L + 63) / 64;                       // upper bound of a CTA's walk
    long s = (target + ctas - 1) / ctas;
    s = s < 8 ? s : 8;
    while (s > 1 && key_tiles / s < 16) --s;                     // at least 16 key tiles per slice
    return (int)s;
}

TcWorkspace tc_workspace_layout(const hyq_attn_args& a) {
    TcWorkspace w{};
    size_t off = 0;
    auto take = [&](size_t bytes) { const size_t o = off; off += align_up(bytes, 1024); return o; };
    const size_t kv_elems = (size_t)a.B * a.Hkv * a.L * HYQ_D, q_elems = (size_t)a.B * a.Hq * query_rows(a) * HYQ_D;
    w.mask_words = (a.L + 127) / 128 * 4;
    w.vl_bits = take((size_t)a.B * a.Hq * w.mask_words * 4);
    w.v16 = take(kv_elems * 2);
    w.vh16 = take(kv_elems * 2);
    w.kvl = take((size_t)a.B * a.Hq * (a.k > 0 ? a.k : 1) * HYQ_D * 2);
    w.vvl = take((size_t)a.B * a.Hq * (a.k > 0 ? a.k : 1) * HYQ_D * 2);
    const bool int4 = a.q_format == HYQ_FMT_INT4;
    w.q8 = int4 ? take(q_elems) : 0;
    w.k8 = int4 ? take(kv_elems) : 0;
    w.vl_tiles = (a.q_format != HYQ_FMT_INT8 && a.k > 0) ? take((size_t)a.B * a.Hq * (w.mask_words / 2) * VL_TILE_BYTES) : 0;
    w.splits = tc_key_splits(a);
    w.redo = take((1 + 3 * (size_t)((query_rows(a) + 255) / 256) * w.splits * a.Hq * a.B) * 4);
    const size_t rows = (size_t)a.B * a.Hq * query_rows(a);
    w.part_o = w.splits > 1 ? take((size_t)w.splits * rows * HYQ_D * 4) : 0;
    w.part_ml = w.splits > 1 ? take((size_t)w.splits * rows * 2 * 4) : 0;
    w.total = off;
    return w;
}

int launch_tc_prepass(const hyq_attn_args& a, const TcWorkspace& w, cudaStream_t st) {
    char* base = static_cast<char*>(a.workspace);
    const long n_heads = (long)a.B * a.Hq;
    uint32_t* bits = reinterpret_cast<uint32_t*>(base + w.vl_bits);
    if (launch_vl_bitmask(a.vl_idx, n_heads, a.k, a.L, w.mask_words, bits, st) != HYQ_OK) return HYQ_ERR_CUDA;
    if (a.k > 0) {
        const long n = n_heads * a.k;
        gather_vl_kernel<<<(unsigned)((n * 32 + 255) / 256), 256, 0, st>>>(
            static_cast<const __nv_bfloat16*>(a.k_), static_cast<const __nv_bfloat16*>(a.v), a.vl_idx, a.Hq, a.Hkv, a.L,
            a.k, n, reinterpret_cast<__nv_bfloat16*>(base + w.kvl), reinterpret_cast<__half*>(base + w.vvl));
        if (launch_status() != HYQ_OK) return HYQ_ERR_CUDA;
    }
    if (a.q_format != HYQ_FMT_INT8 && a.k > 0) {
        uint8_t* tiles = reinterpret_cast<uint8_t*>(base + w.vl_tiles);
        if (cudaMemsetAsync(tiles, 0, (size_t)n_heads * (w.mask_words / 2) * VL_TILE_BYTES, st) != cudaSuccess) return HYQ_ERR_CUDA;
        const long n = n_heads * a.k;
        vl_mask_tiles_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(a.vl_idx, n_heads, a.k, a.L, w.mask_words / 2, tiles);
        if (launch_status() != HYQ_OK) return HYQ_ERR_CUDA;
    }
    const int nb = (a.L + a.block_tokens - 1) / a.block_tokens;
    const long n_vec = (long)a.B * a.Hkv * a.L * (HYQ_D / 8);
    const unsigned vgrid = (unsigned)((n_vec + 255) / 256);
    if (a.v_format == HYQ_FMT_INT8)
        v_to_fp16_kernel<HYQ_FMT_INT8><<<vgrid, 256, 0, st>>>(static_cast<const uint4*>(a.v), static_cast<const uint2*>(a.v_codes),
            a.v_scales, a.L, nb, a.block_tokens, n_vec, reinterpret_cast<uint4*>(base + w.v16), reinterpret_cast<uint4*>(base + w.vh16));
    else
        v_to_fp16_kernel<HYQ_FMT_FP8_E4M3><<<vgrid, 256, 0, st>>>(static_cast<const uint4*>(a.v), static_cast<const uint2*>(a.v_codes),
            a.v_scales, a.L, nb, a.block_tokens, n_vec, reinterpret_cast<uint4*>(base + w.v16), reinterpret_cast<uint4*>(base + w.vh16));
    if (launch_status() != HYQ_OK) return HYQ_ERR_CUDA;
    if (a.q_format == HYQ_FMT_INT4) {
        const long qw = (long)a.B * a.Hq * query_rows(a) * (HYQ_D / 8), kw = (long)a.B * a.Hkv * a.L * (HYQ_D / 8);
        int4_to_e4m3_kernel<<<(unsigned)((qw + 255) / 256), 256, 0, st>>>(static_cast<const uint32_t*>(a.q_codes), qw,
                                                                        reinterpret_cast<uint2*>(base + w.q8));
        int4_to_e4m3_kernel<<<(unsigned)((kw + 255) / 256), 256, 0, st>>>(static_cast<const uint32_t*>(a.k_codes), kw,
                                                                        reinterpret_cast<uint2*>(base + w.k8));
        if (launch_status() != HYQ_OK) return HYQ_ERR_CUDA;
    }
    return HYQ_OK;
}

}  // namespace hyq
