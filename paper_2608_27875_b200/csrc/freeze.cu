// Freeze (Algorithm 4): builds the hybrid KV cache of the decode stage from the prefill cache.
//
// Two kernels, both HBM-bound and read-once / write-once:
//   gather_rows_kernel     copies the vertical rows (by index) and the window rows (a slice) as bf16;
//   freeze_quantize_kernel one CTA per group of G (32, 64 or 128) COMPACTED rows of one (b, kv head) and one tensor
//                          (K or V): finds the source rows (the complement of the ascending vertical
//                          set, by binary search), quantizes the G x 128 group to INT4 with the
//                          arithmetic of the per-tile quantizer (fp32, one rounding per operation), and
//                          writes K row-major and V in the fragment-major tile layout the decode kernel
//                          loads straight into matrix-instruction operand registers.
#include <cuda_fp8.h>

#include "common.cuh"
#include "decode_common.cuh"

namespace hyq {

constexpr int FRZ_THREADS = 128;     // gather kernel; the quantizer runs 2 * G threads (64 elements per thread)
constexpr int FRZ_QTHREADS_PER_SM = 896;   // quantizer threads resident per SM the register budget is set for (7 CTAs of 128)

// Source position of compacted row p: p + j with j the number of vertical indices below it,
// i.e. the smallest j with idx[j] - j > p (idx ascending, so idx[j] - j never decreases).
__device__ __forceinline__ int source_row(const int32_t* __restrict__ idx, int k, int p) {
    int lo = 0, hi = k;
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (__ldg(idx + mid) - mid > p) hi = mid; else lo = mid + 1;
    }
    return p + lo;
}

__global__ void __launch_bounds__(FRZ_THREADS)
gather_rows_kernel(const uint4* __restrict__ k_, const uint4* __restrict__ v, const int32_t* __restrict__ idx,
                   int N, int W, int k_vl, long sK, long sW, uint4* __restrict__ k_vl_out, uint4* __restrict__ v_vl_out,
                   uint4* __restrict__ k_win, uint4* __restrict__ v_win) {
    const long head = blockIdx.y;
    const int o = blockIdx.x * 8 + (threadIdx.x >> 4);
    const int c = threadIdx.x & 15;                       // 16 x 16 bytes = one 256-byte row
    if (o >= k_vl + W) return;
    const int P = N - W;
    const bool vl = o < k_vl;
    // (a vertical index outside [0, N) is clamped: it then names a wrong row instead of memory outside the tensor)
    const int src = vl ? min(max(__ldg(idx + head * k_vl + o), 0), N - 1) : P + (o - k_vl);
    const long s = (head * N + src) * 16 + c;
    const long d = vl ? (head * sK + o) * 16 + c : (head * sW + (o - k_vl)) * 16 + c;
    (vl ? k_vl_out : k_win)[d] = __ldg(k_ + s);
    (vl ? v_vl_out : v_win)[d] = __ldg(v + s);
}

template <int G, int FMT>
__global__ void __launch_bounds__(2 * G, FRZ_QTHREADS_PER_SM / (2 * G))
freeze_quantize_kernel(const uint4* __restrict__ k_, const uint4* __restrict__ v, const int32_t* __restrict__ idx,
                       int N, int k_vl, int nQ, long nQp, uint8_t* __restrict__ kq, uint8_t* __restrict__ vq,
                       float* __restrict__ ks, float* __restrict__ vs) {
    const int grp = blockIdx.x;
    const long head = blockIdx.y;
    const bool is_v = blockIdx.z == 1;
    const uint4* x = (is_v ? v : k_) + head * N * 16;
    const int32_t* hidx = idx + head * k_vl;

    constexpr int NT = 2 * G;                                  // threads of this CTA
    __shared__ int src[G];
    __shared__ float warp_max[NT / 32];
    constexpr bool FMT8 = FMT != HYQ_FMT_INT4;                 // byte-wide codes (INT8 or FP8 e4m3)
    constexpr int ROW_BYTES = FMT8 ? HYQ_D : HYQ_D / 2;        // code bytes per row
    constexpr int TILE_BYTES = 16 * ROW_BYTES;                 // one 16-row V tile
    constexpr float CB = FMT == HYQ_FMT_INT8 ? 127.0f : FMT == HYQ_FMT_FP8_E4M3 ? 448.0f : 7.0f;
    // V codes are staged row-major with 16 bytes of padding per row, so that both the row-wise stores and the
    // word loads of the fragment-major write-out below spread over the banks
    constexpr int VSTRIDE = ROW_BYTES + 16;
    __shared__ __align__(16) uint8_t vstage[G * VSTRIDE];
    // Source rows of the group's G compacted rows in two dependent memory round trips and a short scan: every warp
    // finds j0 = the number of vertical rows before the group's first row by the same 32-way search (no hand-over
    // between warps), then each row walks on from j0 through the few indices that fall inside the group (a row
    // behind a long run of vertical rows falls back to the binary search).
    const int p0 = grp * G;
    int j0;
    {
        const int ln = threadIdx.x & 31;
        int lo = 0, hi = k_vl;                              // smallest j in [lo, hi] with idx[j] - j > p0
        while (lo < hi) {
            const int step = (hi - lo + 31) >> 5;
            const int pos = lo + ln * step;
            const bool below = pos < hi && __ldg(hidx + pos) - pos <= p0;      // predicate still false at pos
            const int f = __popc(__ballot_sync(0xffffffffu, below));            // falses form a prefix of the lanes
            const int new_lo = f ? lo + (f - 1) * step + 1 : lo;
            const int new_hi = f == 0 ? lo : (f < 32 && lo + f * step < hi ? lo + f * step : hi);
            lo = new_lo; hi = new_hi;
        }
        j0 = lo;
    }
    if (threadIdx.x < G) {
        const int p = p0 + threadIdx.x;
        int s = -1;
        if (p < nQ) {
            int j = j0, steps = 0;                          // smallest j >= j0 with idx[j] - j > p
            while (j < k_vl && steps < 16 && __ldg(hidx + j) - j <= p) { ++j; ++steps; }
            s = (steps < 16) ? p + j : source_row(hidx, k_vl, p);
            s = min(s, N - 1);                              // (only a malformed index list can reach the clamp)
        }
        src[threadIdx.x] = s;
    }
    __syncthreads();

    uint4 r[4][2];
    float amax = 0.0f;
#pragma unroll
    for (int gi = 0; gi < 4; ++gi) {
        const int u = threadIdx.x + gi * NT;              // 16-channel unit: row u >> 3, channels 16 * (u & 7)
        const int s = src[u >> 3];
        if (s >= 0) {
            r[gi][0] = __ldg(x + (long)s * 16 + (u & 7) * 2);
            r[gi][1] = __ldg(x + (long)s * 16 + (u & 7) * 2 + 1);
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
    if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = amax;
    __syncthreads();
    amax = warp_max[0];
#pragma unroll
    for (int w = 1; w < NT / 32; ++w) amax = fmaxf(amax, warp_max[w]);

    const bool dead = !(amax >= 0x1p-100f);
    const float inv = dead ? 0.0f : __fdiv_rn(CB, amax);
    if (threadIdx.x == 0) (is_v ? vs : ks)[head * (nQp / G) + grp] = dead ? 0.0f : __fdiv_rn(amax, CB);

#pragma unroll
    for (int gi = 0; gi < 4; ++gi) {
        const int u = threadIdx.x + gi * NT;
        const int row = u >> 3, ch0 = (u & 7) * 16;
        const uint32_t* w = reinterpret_cast<const uint32_t*>(&r[gi][0]);
        if (FMT8) {
            uint32_t o[4] = {0u, 0u, 0u, 0u};
#pragma unroll
            for (int m = 0; m < 8; ++m) {
                const float y0 = __fmul_rn(bf16_lo(w[m]), inv), y1 = __fmul_rn(bf16_hi(w[m]), inv);
                uint32_t two;                                // codes of channels 2m (low byte) and 2m + 1
                if (FMT == HYQ_FMT_FP8_E4M3) {
                    two = dead ? 0u : __nv_cvt_float2_to_fp8x2(make_float2(y0, y1), __NV_SATFINITE, __NV_E4M3);   // no -0 in a zero group
                } else {
                    two = (uint32_t)(max(-127, min(127, __float2int_rn(y0))) & 0xFF) |
                          ((uint32_t)(max(-127, min(127, __float2int_rn(y1))) & 0xFF) << 8);
                }
                o[m >> 1] |= (two & 0xFFFFu) << (16 * (m & 1));
            }
            uint4* d4 = is_v ? reinterpret_cast<uint4*>(vstage + row * VSTRIDE + ch0)
                             : reinterpret_cast<uint4*>(kq + ((head * nQp + grp * G + row) * ROW_BYTES + ch0));
            *d4 = make_uint4(o[0], o[1], o[2], o[3]);
        } else {
            uint32_t o[2] = {0u, 0u};
#pragma unroll
            for (int m = 0; m < 8; ++m) {
                const int q0 = max(-7, min(7, __float2int_rn(__fmul_rn(bf16_lo(w[m]), inv))));
                const int q1 = max(-7, min(7, __float2int_rn(__fmul_rn(bf16_hi(w[m]), inv))));
                o[m >> 2] |= (uint32_t)((q0 & 0xF) | ((q1 & 0xF) << 4)) << (8 * (m & 3));
            }
            uint2* d2 = is_v ? reinterpret_cast<uint2*>(vstage + row * VSTRIDE + ch0 / 2)
                             : reinterpret_cast<uint2*>(kq + ((head * nQp + grp * G + row) * ROW_BYTES + ch0 / 2));
            *d2 = make_uint2(o[0], o[1]);
        }
    }
    if (is_v) {
        // Fragment-major write-out (the layouts of vq_byte_offset / vq8_byte_offset): 16-byte piece number 32 * run + l
        // of a tile, l = 4r + j, is made of one 4-byte load from each of the rows 2j, 2j + 1, 2j + 8, 2j + 9 and
        // a 4 x 4 (INT4) or 2 x 2 (byte codes) transpose of their bytes.
        __syncthreads();
        uint4* dst = reinterpret_cast<uint4*>(vq + (head * (nQp / 16) + grp * (G / 16)) * (long)TILE_BYTES);
        constexpr int PIECES = TILE_BYTES / 16;
#pragma unroll
        for (int i = 0; i < (G / 16) * PIECES / NT; ++i) {
            const int o = threadIdx.x + i * NT;
            const int tile = o / PIECES, run = (o % PIECES) >> 5, r = (o & 31) >> 2, j = o & 3;
            const int col = FMT8 ? 64 * (run >> 1) + 8 * r + 4 * (run & 1) : 32 * run + 4 * r;
            const uint8_t* base = vstage + (tile * 16 + 2 * j) * VSTRIDE + col;
            const uint32_t e0 = *reinterpret_cast<const uint32_t*>(base);                  // row 2j
            const uint32_t o0 = *reinterpret_cast<const uint32_t*>(base + VSTRIDE);        // row 2j + 1
            const uint32_t e1 = *reinterpret_cast<const uint32_t*>(base + 8 * VSTRIDE);    // row 2j + 8
            const uint32_t o1 = *reinterpret_cast<const uint32_t*>(base + 9 * VSTRIDE);    // row 2j + 9
            uint4 out;
            if (FMT8) {
                out.x = __byte_perm(e0, o0, 0x5140);
                out.y = __byte_perm(e1, o1, 0x5140);
                out.z = __byte_perm(e0, o0, 0x7362);
                out.w = __byte_perm(e1, o1, 0x7362);
            } else {
                const uint32_t t0 = __byte_perm(e0, e1, 0x5140), t1 = __byte_perm(e0, e1, 0x7362);
                const uint32_t t2 = __byte_perm(o0, o1, 0x5140), t3 = __byte_perm(o0, o1, 0x7362);
                out.x = __byte_perm(t0, t2, 0x5410);
                out.y = __byte_perm(t0, t2, 0x7632);
                out.z = __byte_perm(t1, t3, 0x5410);
                out.w = __byte_perm(t1, t3, 0x7632);
            }
            dst[o] = out;
        }
    }
}

// one new token per sequence: rows [B*Hkv][128] bf16 -> row `row` of every head's staging buffer
__global__ void __launch_bounds__(FRZ_THREADS)
append_rows_kernel(const uint4* __restrict__ k_new, const uint4* __restrict__ v_new, long heads, int row, int Ws,
                   uint4* __restrict__ k_s, uint4* __restrict__ v_s) {
    const long e = (long)blockIdx.x * FRZ_THREADS + threadIdx.x;     // 16 x 16 bytes per head row
    if (e >= heads * 16) return;
    const long head = e >> 4, c = e & 15;
    const long d = (head * Ws + row) * 16 + c;
    k_s[d] = __ldg(k_new + e);
    v_s[d] = __ldg(v_new + e);
}

int launch_cache_append(const void* k_new, const void* v_new, const hyq_kv_cache& c, cudaStream_t st) {
    const long heads = (long)c.B * c.Hkv;
    append_rows_kernel<<<(unsigned)((heads * 16 + FRZ_THREADS - 1) / FRZ_THREADS), FRZ_THREADS, 0, st>>>(
        static_cast<const uint4*>(k_new), static_cast<const uint4*>(v_new), heads, c.n_staging, c.staging_capacity,
        static_cast<uint4*>(c.k_s), static_cast<uint4*>(c.v_s));
    return launch_status();
}

int launch_freeze(const void* k_, const void* v, const int32_t* vl_idx, const hyq_kv_cache& c, cudaStream_t st) {
    const CacheGeo g = cache_geo(c);
    const long heads = (long)c.B * c.Hkv;
    const uint4* k4 = static_cast<const uint4*>(k_);
    const uint4* v4 = static_cast<const uint4*>(v);
    if (c.k + g.W > 0) {
        const dim3 grid((unsigned)((c.k + g.W + 7) / 8), (unsigned)heads);
        gather_rows_kernel<<<grid, FRZ_THREADS, 0, st>>>(k4, v4, vl_idx, c.N, g.W, c.k, g.sK, g.sW, static_cast<uint4*>(c.k_vl),
                                                         static_cast<uint4*>(c.v_vl), static_cast<uint4*>(c.k_win),
                                                         static_cast<uint4*>(c.v_win));
    }
    if (g.nQ > 0) {
        const dim3 grid((unsigned)(g.nQp / c.group), (unsigned)heads, 2);
        auto* kq = static_cast<uint8_t*>(c.kq_codes);
        auto* vq = static_cast<uint8_t*>(c.vq_codes);
#define HYQ_FRZ(G_, F8_) freeze_quantize_kernel<G_, F8_><<<grid, 2 * G_, 0, st>>>(k4, v4, vl_idx, c.N, c.k, (int)g.nQ, g.sQ, kq, vq, c.kq_scales, c.vq_scales)
#define HYQ_FRZ_F(G_) do { if (c.format == HYQ_FMT_INT8) HYQ_FRZ(G_, HYQ_FMT_INT8); else if (c.format == HYQ_FMT_FP8_E4M3) HYQ_FRZ(G_, HYQ_FMT_FP8_E4M3); else HYQ_FRZ(G_, HYQ_FMT_INT4); } while (0)
        if (c.group == 32) HYQ_FRZ_F(32);
        else if (c.group == 64) HYQ_FRZ_F(64);
        else HYQ_FRZ_F(128);
#undef HYQ_FRZ_F
#undef HYQ_FRZ
    }
    return launch_status();
}

}  // namespace hyq
