// Hybrid-precision causal attention (Eq. 6-7), plain CUDA-core version.
//
// A deliberately simple fp32 kernel used to cross-check the tensor-core kernel on the device
// at sizes where a CPU check can only sample rows.  One CTA of 256 threads owns 64 query rows
// of one (b, head) and walks the key tiles (64 keys) in position order with the running
// (m, l, acc) update of Algorithm 2 Stage 3.  For every tile both score kinds are computed
// (bf16 originals in fp32, integer codes with dp4a) and each pair keeps the one of its class:
// full precision when the key is a vertical-line key of the head or i - j < window.
#include <cuda_fp8.h>

#include "attn_common.cuh"

namespace hyq {

constexpr int ST = 64;               // query rows and keys per tile
constexpr int SIMT_THREADS = 256;
constexpr int QK_STRIDE = HYQ_D / 2 + 1;     // words per bf16 row (+1 pad)
constexpr int C_STRIDE = HYQ_D / 4 + 1;      // words per int8 code row (+1 pad)
constexpr int P_STRIDE = ST + 1;
constexpr int V_STRIDE = HYQ_D + 4;

struct SimtSmem {
    uint32_t q[ST * QK_STRIDE];
    uint32_t k[ST * QK_STRIDE];
    uint32_t qc[ST * C_STRIDE];
    uint32_t kc[ST * C_STRIDE];
    float v[ST * V_STRIDE];
    float vh[ST * V_STRIDE];
    float p_fp[ST * P_STRIDE];
    float p_lq[ST * P_STRIDE];
    float q_scale[ST];
    float k_scale[ST];
};

__device__ __forceinline__ float e4m3_to_float(uint8_t code) {
    const __half_raw hr = __nv_cvt_fp8_to_halfraw(code, __NV_E4M3);
    return __half2float(__half(hr));
}

// 8 signed 4-bit codes (one 32-bit word) -> two words of int8 codes
__device__ __forceinline__ void unpack_int4x8(uint32_t w, uint32_t& lo, uint32_t& hi) {
    uint32_t o[2] = {0u, 0u};
#pragma unroll
    for (int n = 0; n < 8; ++n) {
        const int v = ((int)(w << (28 - 4 * n))) >> 28;      // sign-extended nibble n
        o[n >> 2] |= (uint32_t)(v & 0xFF) << ((n & 3) * 8);
    }
    lo = o[0];
    hi = o[1];
}

// stage `rows` code rows (int8, e4m3 bytes, or packed int4 widened to int8) as byte words; rows beyond n_rows are zero
template <int FMT>
__device__ __forceinline__ void stage_codes(uint32_t* dst, const uint8_t* src, int n_rows) {
    constexpr int ROW_WORDS = (FMT == HYQ_FMT_INT4) ? HYQ_D / 8 : HYQ_D / 4;
    for (int e = threadIdx.x; e < ST * ROW_WORDS; e += SIMT_THREADS) {
        const int r = e / ROW_WORDS, c = e % ROW_WORDS;
        const uint32_t w = (r < n_rows) ? reinterpret_cast<const uint32_t*>(src)[(long)r * ROW_WORDS + c] : 0u;
        if (FMT == HYQ_FMT_INT4) {
            unpack_int4x8(w, dst[r * C_STRIDE + 2 * c], dst[r * C_STRIDE + 2 * c + 1]);
        } else {
            dst[r * C_STRIDE + c] = w;
        }
    }
}

__device__ __forceinline__ void stage_bf16(uint32_t* dst, const __nv_bfloat16* src, int n_rows) {
    for (int e = threadIdx.x; e < ST * (HYQ_D / 2); e += SIMT_THREADS) {
        const int r = e / (HYQ_D / 2), c = e % (HYQ_D / 2);
        dst[r * QK_STRIDE + c] = (r < n_rows) ? reinterpret_cast<const uint32_t*>(src)[(long)r * (HYQ_D / 2) + c] : 0u;
    }
}

template <int QK_FMT, int V_FMT>
__global__ void __launch_bounds__(SIMT_THREADS)
attn_simt_kernel(hyq_attn_args a, float alpha, const uint32_t* __restrict__ vl_bits) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    SimtSmem& sm = *reinterpret_cast<SimtSmem*>(smem_raw);
    // L keys; Lq query rows, end-aligned: query row i sits at position i + off
    const int L = a.L, Lq = query_rows(a), off = L - Lq, g = a.Hq / a.Hkv;
    const int bt = a.block_tokens;                       // tokens per quantization block (32, 64 or 128)
    const int nb = (L + bt - 1) / bt, nbq = (Lq + bt - 1) / bt;
    const int i0 = blockIdx.x * ST, h = blockIdx.y, b = blockIdx.z, kvh = h / g;
    const long qhead = (long)b * a.Hq + h, kvhead = (long)b * a.Hkv + kvh;
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    const int n_q = min(ST, Lq - i0);
    constexpr int QK_ROW_BYTES = (QK_FMT == HYQ_FMT_INT4) ? HYQ_D / 2 : HYQ_D;
    const int mask_words = (L + 31) / 32;
    const uint32_t* vl_row = vl_bits + qhead * mask_words;

    stage_bf16(sm.q, static_cast<const __nv_bfloat16*>(a.q) + (qhead * Lq + i0) * HYQ_D, n_q);
    stage_codes<QK_FMT>(sm.qc, static_cast<const uint8_t*>(a.q_codes) + (qhead * Lq + i0) * QK_ROW_BYTES, n_q);
    if (threadIdx.x < ST) sm.q_scale[threadIdx.x] = a.q_scales[qhead * nbq + min(i0 + (int)threadIdx.x, Lq - 1) / bt];

    float m_run[4], l_run[4], acc[4][8];
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        m_run[r] = -INFINITY;
        l_run[r] = 0.0f;
#pragma unroll
        for (int c = 0; c < 8; ++c) acc[r][c] = 0.0f;
    }

    for (int j0 = 0; j0 <= off + i0 + n_q - 1; j0 += ST) {
        const int n_k = min(ST, L - j0);
        __syncthreads();
        stage_bf16(sm.k, static_cast<const __nv_bfloat16*>(a.k_) + (kvhead * L + j0) * HYQ_D, n_k);
        stage_codes<QK_FMT>(sm.kc, static_cast<const uint8_t*>(a.k_codes) + (kvhead * L + j0) * QK_ROW_BYTES, n_k);
        if (threadIdx.x < ST) sm.k_scale[threadIdx.x] = a.k_scales[kvhead * nb + min(j0 + (int)threadIdx.x, L - 1) / bt];
        for (int e = threadIdx.x; e < ST * HYQ_D; e += SIMT_THREADS) {
            const int r = e / HYQ_D, c = e % HYQ_D;
            float vf = 0.0f, vq = 0.0f;
            if (r < n_k) {
                vf = __bfloat162float(static_cast<const __nv_bfloat16*>(a.v)[(kvhead * L + j0 + r) * HYQ_D + c]);
                const uint8_t code = static_cast<const uint8_t*>(a.v_codes)[(kvhead * L + j0 + r) * HYQ_D + c];
                const float sv = a.v_scales[kvhead * nb + (j0 + r) / bt];
                vq = ((V_FMT == HYQ_FMT_INT8) ? (float)(int8_t)code : e4m3_to_float(code)) * sv;
            }
            sm.v[r * V_STRIDE + c] = vf;
            sm.vh[r * V_STRIDE + c] = vq;
        }
        __syncthreads();

        // scores of the 4x4 pairs (rows ty*4.., keys tx*4..) in both classes
        float s_fp[4][4];
        int s_lq[4][4];
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int c = 0; c < 4; ++c) { s_fp[r][c] = 0.0f; s_lq[r][c] = 0; }
        for (int w = 0; w < HYQ_D / 2; ++w) {
            float ql[4], qh[4], kl[4], kh[4];
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                const uint32_t qw = sm.q[(ty * 4 + r) * QK_STRIDE + w], kw = sm.k[(tx * 4 + r) * QK_STRIDE + w];
                ql[r] = bf16_lo(qw); qh[r] = bf16_hi(qw); kl[r] = bf16_lo(kw); kh[r] = bf16_hi(kw);
            }
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
                for (int c = 0; c < 4; ++c) s_fp[r][c] = fmaf(qh[r], kh[c], fmaf(ql[r], kl[c], s_fp[r][c]));
        }
        float s_lqf[4][4];                               // e4m3 codes: the code products are summed as floats
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int c = 0; c < 4; ++c) s_lqf[r][c] = 0.0f;
        for (int w = 0; w < HYQ_D / 4; ++w) {
            int qv[4], kv[4];
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                qv[r] = (int)sm.qc[(ty * 4 + r) * C_STRIDE + w];
                kv[r] = (int)sm.kc[(tx * 4 + r) * C_STRIDE + w];
            }
            if (QK_FMT == HYQ_FMT_FP8_E4M3) {
                float qf[4][4], kf[4][4];
#pragma unroll
                for (int r = 0; r < 4; ++r)
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        qf[r][e] = e4m3_to_float((uint8_t)((uint32_t)qv[r] >> (8 * e)));
                        kf[r][e] = e4m3_to_float((uint8_t)((uint32_t)kv[r] >> (8 * e)));
                    }
#pragma unroll
                for (int r = 0; r < 4; ++r)
#pragma unroll
                    for (int c = 0; c < 4; ++c)
#pragma unroll
                        for (int e = 0; e < 4; ++e) s_lqf[r][c] = fmaf(qf[r][e], kf[c][e], s_lqf[r][c]);
            } else {
#pragma unroll
                for (int r = 0; r < 4; ++r)
#pragma unroll
                    for (int c = 0; c < 4; ++c) s_lq[r][c] = __dp4a(qv[r], kv[c], s_lq[r][c]);
            }
        }

        // class selection, masks, online softmax
        bool fp[4][4];
        float s[4][4];
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const int i = off + i0 + ty * 4 + r;        // position of the query row among the keys
            float mx = m_run[r];
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const int j = j0 + tx * 4 + c;
                const bool valid = (j <= i) && (j < L) && (i < L);       // (i < L <=> the row exists)
                const bool is_vl = valid && ((vl_row[j >> 5] >> (j & 31)) & 1u);
                fp[r][c] = is_vl || (a.window_mode == HYQ_WINDOW_FIXED_TAIL ? (j >= L - a.window) : (i - j < a.window));
                const float code_dot = (QK_FMT == HYQ_FMT_FP8_E4M3) ? s_lqf[r][c] : (float)s_lq[r][c];
                const float lq = code_dot * sm.q_scale[ty * 4 + r] * sm.k_scale[tx * 4 + c] * alpha;
                s[r][c] = valid ? (fp[r][c] ? s_fp[r][c] * alpha : lq) : -INFINITY;
                mx = fmaxf(mx, s[r][c]);
            }
#pragma unroll
            for (int o = 8; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
            const float m_new = mx;                      // finite from the first tile on (key 0 is valid for every row)
            const float corr = (m_run[r] == -INFINITY) ? 0.0f : expf(m_run[r] - m_new);
            float rs = 0.0f;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const float p = (s[r][c] == -INFINITY || m_new == -INFINITY) ? 0.0f : expf(s[r][c] - m_new);
                rs += p;
                sm.p_fp[(ty * 4 + r) * P_STRIDE + tx * 4 + c] = fp[r][c] ? p : 0.0f;
                sm.p_lq[(ty * 4 + r) * P_STRIDE + tx * 4 + c] = fp[r][c] ? 0.0f : p;
            }
#pragma unroll
            for (int o = 8; o > 0; o >>= 1) rs += __shfl_xor_sync(0xffffffffu, rs, o);
            l_run[r] = l_run[r] * corr + rs;
            m_run[r] = m_new;
#pragma unroll
            for (int c = 0; c < 8; ++c) acc[r][c] *= corr;
        }
        __syncthreads();

        // acc += P_fp . V + P_lq . V^   (rows ty*4.., channels tx*8..)
        for (int j = 0; j < ST; ++j) {
            float vf[8], vq[8];
#pragma unroll
            for (int c = 0; c < 8; ++c) { vf[c] = sm.v[j * V_STRIDE + tx * 8 + c]; vq[c] = sm.vh[j * V_STRIDE + tx * 8 + c]; }
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                const float pf = sm.p_fp[(ty * 4 + r) * P_STRIDE + j], pq = sm.p_lq[(ty * 4 + r) * P_STRIDE + j];
#pragma unroll
                for (int c = 0; c < 8; ++c) acc[r][c] = fmaf(pq, vq[c], fmaf(pf, vf[c], acc[r][c]));
            }
        }
    }

#pragma unroll
    for (int r = 0; r < 4; ++r) {
        const int i = i0 + ty * 4 + r;
        if (i >= Lq) continue;
        const float inv = 1.0f / l_run[r];
        if (a.out_dtype == 1) {
            float* o = static_cast<float*>(a.out) + (qhead * Lq + i) * HYQ_D + tx * 8;
#pragma unroll
            for (int c = 0; c < 8; ++c) o[c] = acc[r][c] * inv;
        } else {
            __nv_bfloat16* o = static_cast<__nv_bfloat16*>(a.out) + (qhead * Lq + i) * HYQ_D + tx * 8;
#pragma unroll
            for (int c = 0; c < 8; ++c) o[c] = __float2bfloat16_rn(acc[r][c] * inv);
        }
        if (a.lse && tx == 0) a.lse[qhead * Lq + i] = m_run[r] + logf(l_run[r]);
    }
}

size_t attn_simt_workspace_bytes(const hyq_attn_args& a) {
    return align_up((size_t)a.B * a.Hq * ((a.L + 31) / 32) * 4, 256);
}

int launch_attn_simt(const hyq_attn_args& a, float alpha, cudaStream_t st) {
    const int mask_words = (a.L + 31) / 32;
    const long n_heads = (long)a.B * a.Hq;
    uint32_t* bits = static_cast<uint32_t*>(a.workspace);
    if (launch_vl_bitmask(a.vl_idx, n_heads, a.k, a.L, mask_words, bits, st) != HYQ_OK) return HYQ_ERR_CUDA;
    const dim3 grid((query_rows(a) + ST - 1) / ST, a.Hq, a.B);
    const size_t smem = sizeof(SimtSmem);
    auto run = [&](auto kern) -> int {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return HYQ_ERR_CUDA;
        kern<<<grid, SIMT_THREADS, smem, st>>>(a, alpha, bits);
        return launch_status();
    };
    if (a.q_format == HYQ_FMT_INT8 && a.v_format == HYQ_FMT_INT8) return run(attn_simt_kernel<HYQ_FMT_INT8, HYQ_FMT_INT8>);
    if (a.q_format == HYQ_FMT_INT4 && a.v_format == HYQ_FMT_FP8_E4M3) return run(attn_simt_kernel<HYQ_FMT_INT4, HYQ_FMT_FP8_E4M3>);
    if (a.q_format == HYQ_FMT_FP8_E4M3 && a.v_format == HYQ_FMT_FP8_E4M3) return run(attn_simt_kernel<HYQ_FMT_FP8_E4M3, HYQ_FMT_FP8_E4M3>);
    return HYQ_ERR_UNSUPPORTED;
}

}  // namespace hyq
