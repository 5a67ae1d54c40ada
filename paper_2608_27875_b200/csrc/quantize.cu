// Per-tile symmetric quantization (Algorithm 2, Stage 2).
//
// One CTA of 2 * BT threads owns one tile of BT (32, 64 or 128) tokens x 128 channels: contiguous bf16
// (16 KB for the default 64 tokens).  Each thread keeps its 64 elements in registers (4 groups of 16
// consecutive channels, 32-byte loads), the tile absmax is a warp-shuffle reduction plus one
// shared-memory step across the 4 warps, and the codes leave as 16-byte (8-bit formats) or
// 8-byte (INT4) vector stores.  The tile is read once and written once: HBM-bound.
//
// Arithmetic is fp32 with one IEEE rounding per operation (no FMA contraction, no fast-math):
//   scale = absmax / c ; inv = c / absmax ; code = rint(x * inv) clamped, or e4m3(x * inv).
#include <cuda_fp8.h>

#include "common.cuh"

namespace hyq {

constexpr int QUANT_GROUPS = 4;                       // groups of 16 elements per thread

template <int FMT, int BT>
__global__ void __launch_bounds__(2 * BT)
quantize_tiles_kernel(const uint4* __restrict__ x, int L, int nb, uint8_t* __restrict__ codes,
                      float* __restrict__ scales) {
    constexpr int QUANT_THREADS = 2 * BT;
    const long tile = blockIdx.x;                     // (b*H + h) * nb + n
    const long head = tile / nb;
    const int n = (int)(tile - head * nb);
    const int t0 = n * BT;
    const int tokens = min(BT, L - t0);
    const int n_elems = tokens * HYQ_D;
    const long elem0 = (head * L + t0) * (long)HYQ_D;
    const uint4* src = x + elem0 / 8;

    uint4 r[QUANT_GROUPS][2];
    float amax = 0.0f;
#pragma unroll
    for (int gi = 0; gi < QUANT_GROUPS; ++gi) {
        const int e = (threadIdx.x + gi * QUANT_THREADS) * 16;
        if (e < n_elems) {
            r[gi][0] = __ldg(src + e / 8);
            r[gi][1] = __ldg(src + e / 8 + 1);
        } else {
            r[gi][0] = make_uint4(0, 0, 0, 0);
            r[gi][1] = make_uint4(0, 0, 0, 0);
        }
        const uint32_t* w = reinterpret_cast<const uint32_t*>(&r[gi][0]);
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            amax = fmaxf(amax, fabsf(bf16_lo(w[c])));
            amax = fmaxf(amax, fabsf(bf16_hi(w[c])));
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    __shared__ float warp_max[QUANT_THREADS / 32];
    if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = amax;
    __syncthreads();
    amax = warp_max[0];
#pragma unroll
    for (int w = 1; w < QUANT_THREADS / 32; ++w) amax = fmaxf(amax, warp_max[w]);

    constexpr float c = (FMT == HYQ_FMT_INT8) ? 127.0f : (FMT == HYQ_FMT_FP8_E4M3) ? 448.0f : 7.0f;
    const bool dead = !(amax >= 0x1p-100f);
    const float inv = dead ? 0.0f : __fdiv_rn(c, amax);
    if (threadIdx.x == 0) scales[tile] = dead ? 0.0f : __fdiv_rn(amax, c);

    constexpr int ROW_BYTES = (FMT == HYQ_FMT_INT4) ? HYQ_D / 2 : HYQ_D;
    uint8_t* dst = codes + (head * L + t0) * (long)ROW_BYTES;
#pragma unroll
    for (int gi = 0; gi < QUANT_GROUPS; ++gi) {
        const int e = (threadIdx.x + gi * QUANT_THREADS) * 16;
        if (e >= n_elems) continue;
        const uint32_t* w = reinterpret_cast<const uint32_t*>(&r[gi][0]);
        if (FMT == HYQ_FMT_FP8_E4M3) {
            uint32_t o[4];
#pragma unroll
            for (int c4 = 0; c4 < 4; ++c4) {
                const float y0 = __fmul_rn(bf16_lo(w[2 * c4]), inv), y1 = __fmul_rn(bf16_hi(w[2 * c4]), inv);
                const float y2 = __fmul_rn(bf16_lo(w[2 * c4 + 1]), inv), y3 = __fmul_rn(bf16_hi(w[2 * c4 + 1]), inv);
                const uint32_t lo = __nv_cvt_float2_to_fp8x2(make_float2(y0, y1), __NV_SATFINITE, __NV_E4M3);
                const uint32_t hi = __nv_cvt_float2_to_fp8x2(make_float2(y2, y3), __NV_SATFINITE, __NV_E4M3);
                o[c4] = dead ? 0u : (lo | (hi << 16));      // an all-zero tile has all-zero codes (no -0)
            }
            *reinterpret_cast<uint4*>(dst + e) = make_uint4(o[0], o[1], o[2], o[3]);
        } else {
            int q[16];
#pragma unroll
            for (int c2 = 0; c2 < 8; ++c2) {
                q[2 * c2] = max(-(int)c, min((int)c, __float2int_rn(__fmul_rn(bf16_lo(w[c2]), inv))));
                q[2 * c2 + 1] = max(-(int)c, min((int)c, __float2int_rn(__fmul_rn(bf16_hi(w[c2]), inv))));
            }
            if (FMT == HYQ_FMT_INT8) {
                uint32_t o[4];
#pragma unroll
                for (int c4 = 0; c4 < 4; ++c4)
                    o[c4] = (uint32_t)(q[4 * c4] & 0xFF) | ((uint32_t)(q[4 * c4 + 1] & 0xFF) << 8) |
                            ((uint32_t)(q[4 * c4 + 2] & 0xFF) << 16) | ((uint32_t)(q[4 * c4 + 3] & 0xFF) << 24);
                *reinterpret_cast<uint4*>(dst + e) = make_uint4(o[0], o[1], o[2], o[3]);
            } else {
                uint32_t o[2] = {0u, 0u};
#pragma unroll
                for (int c16 = 0; c16 < 16; ++c16) o[c16 >> 3] |= (uint32_t)(q[c16] & 0xF) << ((c16 & 7) * 4);
                *reinterpret_cast<uint2*>(dst + e / 2) = make_uint2(o[0], o[1]);
            }
        }
    }
}

template <int BT>
static int launch_quantize_bt(const uint4* xs, long tiles, int L, int nb, int format, uint8_t* cs, float* scales, cudaStream_t st) {
    const dim3 grid((unsigned)tiles), block(2 * BT);
    switch (format) {
        case HYQ_FMT_INT8: quantize_tiles_kernel<HYQ_FMT_INT8, BT><<<grid, block, 0, st>>>(xs, L, nb, cs, scales); break;
        case HYQ_FMT_FP8_E4M3: quantize_tiles_kernel<HYQ_FMT_FP8_E4M3, BT><<<grid, block, 0, st>>>(xs, L, nb, cs, scales); break;
        case HYQ_FMT_INT4: quantize_tiles_kernel<HYQ_FMT_INT4, BT><<<grid, block, 0, st>>>(xs, L, nb, cs, scales); break;
        default: return HYQ_ERR_UNSUPPORTED;
    }
    return launch_status();
}

int launch_quantize(const void* x, long n_heads, int L, int block_tokens, int format, void* codes, float* scales, cudaStream_t st) {
    const int nb = (L + block_tokens - 1) / block_tokens;
    const long tiles = n_heads * nb;
    if (tiles <= 0) return HYQ_OK;
    if (tiles > 0x7fffffffL) return HYQ_ERR_INVALID_ARG;
    const uint4* xs = static_cast<const uint4*>(x);
    uint8_t* cs = static_cast<uint8_t*>(codes);
    switch (block_tokens) {
        case 32: return launch_quantize_bt<32>(xs, tiles, L, nb, format, cs, scales, st);
        case 64: return launch_quantize_bt<64>(xs, tiles, L, nb, format, cs, scales, st);
        case 128: return launch_quantize_bt<128>(xs, tiles, L, nb, format, cs, scales, st);
        default: return HYQ_ERR_UNSUPPORTED;
    }
}

}  // namespace hyq
