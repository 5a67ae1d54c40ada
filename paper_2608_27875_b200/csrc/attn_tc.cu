// Fused hybrid-precision causal attention (Eq. 6-7; Algorithm 2, Stage 3) on the 5th-generation
// tensor cores: TMA -> shared memory -> tcgen05.mma -> TMEM, one online softmax over three passes.
//
// One CTA owns 128 query rows of one (b, query head) and walks key tiles of 128:
//   pass A  low-bit keys   j <= i - W, j not vertical   S = Qc.Kc^T  (kind::i8, or kind::f8f6f4 on
//                                                       INT4 codes widened to e4m3), V^ in fp16
//   pass B  vertical keys  gathered per query head, ascending, idx <= i - W   S = Q.Kvl^T (bf16)
//   pass C  window keys    i - W < j <= i                                     S = Q.K^T   (bf16)
// All passes feed one running (m, l) per row and one fp32 O accumulator in TMEM; P goes back to
// TMEM as fp16 and is the A operand of the P.V MMA (fp16 x fp16).
//
// Warp roles (192 threads): warps 0-3 softmax (thread r owns query row r = TMEM lane r),
// warp 4 lane 0 issues TMA loads, warp 5 lane 0 issues MMAs.  S is double-buffered in TMEM so that
// Q.K^T of tile t+1 runs under the softmax of tile t.  Every mbarrier wait is bounded; when one
// expires the CTA records HYQ_ERR_TIMEOUT in the status word and unwinds.
#include <cuda_fp16.h>

#include "attn_common.cuh"
#include "sm100.cuh"

namespace hyq {
using namespace sm100;

constexpr int BM = 128, BN = 128;
constexpr int TC_THREADS = 192;
constexpr long long WAIT_LIMIT = 4000000000LL;      // SM clocks (~2 s): far beyond any legitimate wait

constexpr uint32_t SQ_OFF = 0, SQC_OFF = 32768, SK_OFF = 49152, SV_OFF = SK_OFF + 2 * 32768;
constexpr uint32_t TILE_SMEM = SV_OFF + 2 * 32768;                  // 180224
constexpr uint32_t TC_SMEM_BYTES = TILE_SMEM + 1024;                // + slack for 1024-byte alignment

constexpr uint32_t TM_S0 = 0, TM_S1 = 128, TM_O = 256, TM_COLS = 512;

struct TcMaps {
    CUtensorMap q, k, qc, kc, v16, vh16, kvl, vvl;
};

struct TcParams {
    int B, Hq, Hkv, L, window, k, nb, mask_words;
    int lowbit_fp8;              // 1: low-bit codes are e4m3 bytes (kind::f8f6f4), 0: int8 (kind::i8)
    int out_fp32;
    float scale_log2;            // softmax_scale * log2(e)
    const float* q_scales;
    const float* k_scales;
    const int32_t* vl_idx;
    const uint32_t* vl_bits;
    void* out;
    float* lse;
    int32_t* status;
};

struct TcBarriers {
    uint64_t q_full, k_full[2], k_free[2], v_full[2], v_free[2], s_full[2], p_full[2], o_done;
};

__device__ __forceinline__ float ex2f(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// number of entries of the ascending list idx[0..k) that are <= v
__device__ __forceinline__ int count_le(const int32_t* __restrict__ idx, int k, int v) {
    int lo = 0, hi = k;
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (__ldg(idx + mid) <= v) lo = mid + 1; else hi = mid;
    }
    return lo;
}

__global__ void __launch_bounds__(TC_THREADS, 1)
attn_tc_kernel(const __grid_constant__ TcMaps maps, const TcParams p) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    __shared__ TcBarriers bars;
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s, cnt_b_s;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int qt = gridDim.x - 1 - blockIdx.x;               // longest rows first
    const int h = blockIdx.y, b = blockIdx.z;
    const int L = p.L, W = p.window, g = p.Hq / p.Hkv;
    const int qhead = b * p.Hq + h, kvhead = b * p.Hkv + h / g;
    const int i0 = qt * BM, i1 = min(i0 + BM - 1, L - 1);
    const int32_t* idx_row = p.vl_idx + (long)qhead * p.k;

    if (threadIdx.x == 0) {
        mbar_init(&bars.q_full, 1);
        for (int s = 0; s < 2; ++s) {
            mbar_init(&bars.k_full[s], 1);
            mbar_init(&bars.k_free[s], 1);
            mbar_init(&bars.v_full[s], 1);
            mbar_init(&bars.v_free[s], 1);
            mbar_init(&bars.s_full[s], 1);
            mbar_init(&bars.p_full[s], 128);
        }
        mbar_init(&bars.o_done, 1);
        fence_mbar_init();
        abort_s = 0;
        cnt_b_s = (p.k > 0 && i1 - W >= 0) ? count_le(idx_row, p.k, i1 - W) : 0;
    }
    if (warp == 4) {
        tmem_alloc(&tmem_base_s, TM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_base_s;

    // tile schedule: nA low-bit tiles, nB gathered vertical-line tiles, nC window tiles
    const int nA = (i1 - W >= 0) ? (i1 - W) / BN + 1 : 0;
    const int nB = (cnt_b_s + BN - 1) / BN;
    const int tC0 = (W > 0) ? max(0, i0 - W + 1) / BN : 0;
    const int nC = (W > 0) ? i1 / BN - tC0 + 1 : 0;
    const int T = nA + nB + nC;

    volatile int* abort_flag = &abort_s;
    auto fail = [&]() {
        *abort_flag = 1;
        if (p.status) atomicExch(p.status, HYQ_ERR_TIMEOUT);
    };

    if (warp == 4) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            prefetch_tmap(&maps.q);
            prefetch_tmap(&maps.k);
            mbar_arrive_expect_tx(&bars.q_full, 32768 + (nA > 0 ? 16384 : 0));
            tma_load_3d(smem + SQ_OFF, &maps.q, &bars.q_full, 0, i0, qhead);
            tma_load_3d(smem + SQ_OFF + 16384, &maps.q, &bars.q_full, 64, i0, qhead);
            if (nA > 0) tma_load_3d(smem + SQC_OFF, &maps.qc, &bars.q_full, 0, i0, qhead);
            for (int t = 0; t < T && !*abort_flag; ++t) {
                const int s = t & 1, u = t >> 1;
                unsigned char* sk = smem + SK_OFF + s * 32768;
                unsigned char* sv = smem + SV_OFF + s * 32768;
                if (u > 0 && !mbar_wait(&bars.k_free[s], (u - 1) & 1, WAIT_LIMIT)) { fail(); break; }
                if (t < nA) {
                    mbar_arrive_expect_tx(&bars.k_full[s], 16384);
                    tma_load_3d(sk, &maps.kc, &bars.k_full[s], 0, t * BN, kvhead);
                } else {
                    const bool vl = t < nA + nB;
                    const CUtensorMap* m = vl ? &maps.kvl : &maps.k;
                    const int row = vl ? (t - nA) * BN : (tC0 + t - nA - nB) * BN;
                    const int hd = vl ? qhead : kvhead;
                    mbar_arrive_expect_tx(&bars.k_full[s], 32768);
                    tma_load_3d(sk, m, &bars.k_full[s], 0, row, hd);
                    tma_load_3d(sk + 16384, m, &bars.k_full[s], 64, row, hd);
                }
                if (u > 0 && !mbar_wait(&bars.v_free[s], (u - 1) & 1, WAIT_LIMIT)) { fail(); break; }
                {
                    const bool lowbit = t < nA, vl = !lowbit && t < nA + nB;
                    const CUtensorMap* m = lowbit ? &maps.vh16 : (vl ? &maps.vvl : &maps.v16);
                    const int row = lowbit ? t * BN : (vl ? (t - nA) * BN : (tC0 + t - nA - nB) * BN);
                    const int hd = vl ? qhead : kvhead;
                    mbar_arrive_expect_tx(&bars.v_full[s], 32768);
                    tma_load_3d(sv, m, &bars.v_full[s], 0, row, hd);
                    tma_load_3d(sv + 16384, m, &bars.v_full[s], 64, row, hd);
                }
            }
        }
    } else if (warp == 5) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t sq = smem_u32(smem + SQ_OFF), sqc = smem_u32(smem + SQC_OFF);
            const uint32_t idesc_lq = p.lowbit_fp8 ? make_idesc(ACC_F32, FMT_E4M3, FMT_E4M3, 0, 0, BM, BN)
                                                   : make_idesc(ACC_S32, FMT_S8, FMT_S8, 0, 0, BM, BN);
            const uint32_t idesc_qk = make_idesc(ACC_F32, FMT_BF16, FMT_BF16, 0, 0, BM, BN);
            const uint32_t idesc_pv = make_idesc(ACC_F32, FMT_F16, FMT_F16, 0, 1, BM, HYQ_D);
            bool ok = mbar_wait(&bars.q_full, 0, WAIT_LIMIT);
            auto issue_qk = [&](int t) -> bool {
                const int s = t & 1;
                if (!mbar_wait(&bars.k_full[s], (t >> 1) & 1, WAIT_LIMIT)) return false;
                tc_fence_after();
                const uint32_t sk = smem_u32(smem + SK_OFF + s * 32768);
                const uint32_t d = tmem + (s ? TM_S1 : TM_S0);
                if (t < nA) {
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk) {
                        const uint64_t da = make_smem_desc(sqc + kk * 32, 0, 1024), db = make_smem_desc(sk + kk * 32, 0, 1024);
                        if (p.lowbit_fp8) umma_ss_f8f6f4(d, da, db, idesc_lq, kk > 0);
                        else umma_ss_i8(d, da, db, idesc_lq, kk > 0);
                    }
                } else {
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk) {
                        const uint32_t off = (kk >> 2) * 16384 + (kk & 3) * 32;
                        umma_ss_f16(d, make_smem_desc(sq + off, 0, 1024), make_smem_desc(sk + off, 0, 1024), idesc_qk, kk > 0);
                    }
                }
                umma_commit(&bars.s_full[s]);
                umma_commit(&bars.k_free[s]);
                return true;
            };
            if (ok && T > 0) ok = issue_qk(0);
            for (int t = 0; t < T && ok && !*abort_flag; ++t) {
                if (t + 1 < T) ok = issue_qk(t + 1);
                if (!ok) break;
                const int s = t & 1, par = (t >> 1) & 1;
                if (!mbar_wait(&bars.p_full[s], par, WAIT_LIMIT) || !mbar_wait(&bars.v_full[s], par, WAIT_LIMIT)) { ok = false; break; }
                tc_fence_after();
                const uint32_t sv = smem_u32(smem + SV_OFF + s * 32768);
                const uint32_t pa = tmem + (s ? TM_S1 : TM_S0);
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)
                    umma_ts_f16(tmem + TM_O, pa + kk * 8, make_smem_desc(sv + kk * 2048, 16384, 1024), idesc_pv, (t > 0 || kk > 0));
                umma_commit(&bars.o_done);
                umma_commit(&bars.v_free[s]);
            }
            if (!ok) fail();
        }
    } else {
        // ------------------------------------------------------------------ softmax warps
        const int r = threadIdx.x;                      // query row inside the tile = TMEM lane
        const int i = i0 + r;
        const bool row_live = i < L;
        const uint32_t lane_addr = (uint32_t)(warp * 32) << 16;
        const float q_scale = row_live ? __ldg(p.q_scales + (long)qhead * p.nb + i / HYQ_BLOCK_TOKENS) : 0.0f;
        const int cnt_r = (nB > 0 && row_live && i - W >= 0) ? count_le(idx_row, p.k, i - W) : 0;
        const uint32_t* bits_row = p.vl_bits + (long)qhead * p.mask_words;
        float m_run = -INFINITY, l_run = 0.0f;
        bool ok = true;

        for (int t = 0; t < T; ++t) {
            const int s = t & 1;
            // ---- per-tile column bounds and scales
            int lo = 0, hi = -1;
            bool need_range;
            float cs0, cs1;
            uint32_t vlw[4] = {0u, 0u, 0u, 0u};
            if (t < nA) {
                const int j0 = t * BN;
                hi = row_live ? min(i - W - j0, BN - 1) : -1;
                need_range = (j0 + BN - 1 > i0 - W) || (i0 + BM > L);
                const float k0 = __ldg(p.k_scales + (long)kvhead * p.nb + min(2 * t, p.nb - 1));
                const float k1 = __ldg(p.k_scales + (long)kvhead * p.nb + min(2 * t + 1, p.nb - 1));
                cs0 = q_scale * k0 * p.scale_log2;
                cs1 = q_scale * k1 * p.scale_log2;
#pragma unroll
                for (int w = 0; w < 4; ++w)
                    if (j0 / 32 + w < p.mask_words) vlw[w] = __ldg(bits_row + j0 / 32 + w);
            } else if (t < nA + nB) {
                const int c0 = (t - nA) * BN;
                hi = min(cnt_r - c0 - 1, BN - 1);
                need_range = true;
                cs0 = cs1 = p.scale_log2;
            } else {
                const int j0 = (tC0 + t - nA - nB) * BN;
                lo = max(0, i - W + 1 - j0);
                hi = row_live ? min(i - j0, BN - 1) : -1;
                need_range = (j0 + BN - 1 > i0) || (j0 <= i1 - W) || (i0 + BM > L);
                cs0 = cs1 = p.scale_log2;
            }
            const bool any_vl = (vlw[0] | vlw[1] | vlw[2] | vlw[3]) != 0u;
            const bool int_scores = (t < nA) && !p.lowbit_fp8;

            if (!mbar_wait(&bars.s_full[s], (t >> 1) & 1, WAIT_LIMIT)) { ok = false; break; }
            __syncwarp();
            tc_fence_after();
            const uint32_t ts = tmem + (s ? TM_S1 : TM_S0) + lane_addr;

            float x[BN];
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t raw[32];
                tmem_ld32(ts + c * 32, raw);
                tmem_wait_ld();
                const float cs = (c < 2) ? cs0 : cs1;
#pragma unroll
                for (int e = 0; e < 32; ++e)
                    x[c * 32 + e] = (int_scores ? (float)(int)raw[e] : __uint_as_float(raw[e])) * cs;
            }
            if (need_range) {
#pragma unroll
                for (int c = 0; c < BN; ++c) x[c] = (c >= lo && c <= hi) ? x[c] : -INFINITY;
            }
            if (any_vl) {
#pragma unroll
                for (int c = 0; c < BN; ++c) x[c] = ((vlw[c >> 5] >> (c & 31)) & 1u) ? -INFINITY : x[c];
            }
            float mx = x[0];
#pragma unroll
            for (int c = 1; c < BN; ++c) mx = fmaxf(mx, x[c]);
            const float m_new = fmaxf(m_run, mx);
            const float m_use = (m_new == -INFINITY) ? 0.0f : m_new;
            const float alpha = (m_new == m_run) ? 1.0f : ex2f(m_run - m_use);   // m_run = -inf -> 0

            // ---- the previous P.V must have landed before O is rescaled and before P[s] is rewritten
            if (t > 0) {
                if (!mbar_wait(&bars.o_done, (t - 1) & 1, WAIT_LIMIT)) { ok = false; break; }
                __syncwarp();
                tc_fence_after();
                if (__any_sync(0xffffffffu, alpha != 1.0f)) {
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        uint32_t o[32];
                        tmem_ld32(tmem + TM_O + lane_addr + c * 32, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
                        tmem_st32(tmem + TM_O + lane_addr + c * 32, o);
                    }
                }
            }

            float rs = 0.0f;
#pragma unroll
            for (int hlf = 0; hlf < 2; ++hlf) {
                uint32_t pk[32];
#pragma unroll
                for (int e = 0; e < 32; ++e) {
                    const float p0 = ex2f(x[hlf * 64 + 2 * e] - m_use), p1 = ex2f(x[hlf * 64 + 2 * e + 1] - m_use);
                    rs += p0 + p1;
                    const __half2 h2 = __floats2half2_rn(p0, p1);
                    pk[e] = *reinterpret_cast<const uint32_t*>(&h2);
                }
                tmem_st32(ts + hlf * 32, pk);
            }
            l_run = l_run * alpha + rs;
            m_run = m_new;
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(&bars.p_full[s]);
        }

        // ---- epilogue: O / l
        if (ok && T > 0) ok = mbar_wait(&bars.o_done, (T - 1) & 1, WAIT_LIMIT);
        __syncwarp();
        if (ok) {
            tc_fence_after();
            const float inv = (l_run > 0.0f) ? 1.0f / l_run : 0.0f;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t o[32];
                tmem_ld32(tmem + TM_O + lane_addr + c * 32, o);
                tmem_wait_ld();
                if (row_live) {
                    if (p.out_fp32) {
                        float4* dst = reinterpret_cast<float4*>(static_cast<float*>(p.out) + ((long)qhead * L + i) * HYQ_D + c * 32);
#pragma unroll
                        for (int e = 0; e < 8; ++e)
                            dst[e] = make_float4(__uint_as_float(o[4 * e]) * inv, __uint_as_float(o[4 * e + 1]) * inv,
                                                 __uint_as_float(o[4 * e + 2]) * inv, __uint_as_float(o[4 * e + 3]) * inv);
                    } else {
                        uint4* dst = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(p.out) + ((long)qhead * L + i) * HYQ_D + c * 32);
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            uint32_t w[4];
#pragma unroll
                            for (int q2 = 0; q2 < 4; ++q2) {
                                const __nv_bfloat162 b2 = __floats2bfloat162_rn(__uint_as_float(o[8 * e + 2 * q2]) * inv,
                                                                                __uint_as_float(o[8 * e + 2 * q2 + 1]) * inv);
                                w[q2] = *reinterpret_cast<const uint32_t*>(&b2);
                            }
                            dst[e] = make_uint4(w[0], w[1], w[2], w[3]);
                        }
                    }
                }
            }
            if (p.lse && row_live) p.lse[(long)qhead * L + i] = (m_run + log2f(l_run)) * 0.6931471805599453f;
        } else {
            fail();
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 4) {
        __syncwarp();
        tmem_dealloc(tmem, TM_COLS);
    }
}

// ---------------------------------------------------------------------------------------------
size_t attn_tc_workspace_bytes(const hyq_attn_args& a) { return tc_workspace_layout(a).total; }

int launch_attn_tc(const hyq_attn_args& a, float alpha, cudaStream_t st) {
    const TcWorkspace w = tc_workspace_layout(a);
    const int rc = launch_tc_prepass(a, w, st);
    if (rc != HYQ_OK) return rc;
    char* base = static_cast<char*>(a.workspace);
    const bool int4 = a.q_format == HYQ_FMT_INT4;
    const uint64_t qh = (uint64_t)a.B * a.Hq, kvh = (uint64_t)a.B * a.Hkv, L = a.L;
    const uint64_t kk = a.k > 0 ? a.k : 1;

    TcMaps maps;
    bool ok = true;
    ok &= make_tmap_3d(&maps.q, a.q, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, HYQ_D, L, qh, 64, BM);
    ok &= make_tmap_3d(&maps.k, a.k_, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, HYQ_D, L, kvh, 64, BN);
    ok &= make_tmap_3d(&maps.qc, int4 ? (const void*)(base + w.q8) : a.q_codes, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, HYQ_D, L, qh, 128, BM);
    ok &= make_tmap_3d(&maps.kc, int4 ? (const void*)(base + w.k8) : a.k_codes, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, HYQ_D, L, kvh, 128, BN);
    ok &= make_tmap_3d(&maps.v16, base + w.v16, CU_TENSOR_MAP_DATA_TYPE_UINT16, 2, HYQ_D, L, kvh, 64, BN);
    ok &= make_tmap_3d(&maps.vh16, base + w.vh16, CU_TENSOR_MAP_DATA_TYPE_UINT16, 2, HYQ_D, L, kvh, 64, BN);
    ok &= make_tmap_3d(&maps.kvl, base + w.kvl, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, HYQ_D, kk, qh, 64, BN);
    ok &= make_tmap_3d(&maps.vvl, base + w.vvl, CU_TENSOR_MAP_DATA_TYPE_UINT16, 2, HYQ_D, kk, qh, 64, BN);
    if (!ok) return HYQ_ERR_CUDA;

    TcParams p{};
    p.B = a.B; p.Hq = a.Hq; p.Hkv = a.Hkv; p.L = a.L; p.window = a.window; p.k = a.k;
    p.nb = (a.L + HYQ_BLOCK_TOKENS - 1) / HYQ_BLOCK_TOKENS;
    p.mask_words = w.mask_words;
    p.lowbit_fp8 = int4 ? 1 : 0;
    p.out_fp32 = a.out_dtype == 1;
    p.scale_log2 = alpha * 1.4426950408889634f;
    p.q_scales = a.q_scales; p.k_scales = a.k_scales; p.vl_idx = a.vl_idx;
    p.vl_bits = reinterpret_cast<const uint32_t*>(base + w.vl_bits);
    p.out = a.out; p.lse = a.lse; p.status = a.status_word;

    if (cudaFuncSetAttribute(attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)TC_SMEM_BYTES) != cudaSuccess)
        return HYQ_ERR_CUDA;
    const dim3 grid((a.L + BM - 1) / BM, a.Hq, a.B);
    if (a.ev_kernel_start && cudaEventRecord(static_cast<cudaEvent_t>(a.ev_kernel_start), st) != cudaSuccess) return HYQ_ERR_CUDA;
    attn_tc_kernel<<<grid, TC_THREADS, TC_SMEM_BYTES, st>>>(maps, p);
    if (launch_status() != HYQ_OK) return HYQ_ERR_CUDA;
    if (a.ev_kernel_stop && cudaEventRecord(static_cast<cudaEvent_t>(a.ev_kernel_stop), st) != cudaSuccess) return HYQ_ERR_CUDA;
    return HYQ_OK;
}

}  // namespace hyq
