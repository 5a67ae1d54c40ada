// Fused hybrid-precision causal attention (Eq. 6-7; Algorithm 2, Stage 3) on the 5th-generation
// tensor cores: TMA -> shared memory -> tcgen05.mma -> TMEM, one online softmax over three passes.
//
// One CTA owns 256 query rows (two 128-row tiles) of one (b, query head) and walks key tiles of 128:
//   pass A  low-bit keys   j <= i - W, j not vertical   S = Qc.Kc^T  (kind::i8, or kind::f8f6f4 on
//                                                       INT4 codes widened to e4m3), V^ in fp16
//   pass B  vertical keys  gathered per query head, ascending, idx <= i - W   S = Q.Kvl^T (bf16)
//   pass C  window keys    i - W < j <= i                                     S = Q.K^T   (bf16)
// All passes feed one running (m, l) per row and one fp32 O accumulator per query tile in TMEM; P goes
// back to TMEM as fp16 (over the S columns it was computed from) and is the A operand of the P.V
// MMA (fp16 x fp16).  K/V tiles are loaded once and used by both query tiles.
//
// Warp roles (320 threads): warps 0-3 and 4-7 are the softmax groups of query tile 0 and 1 (thread r
// owns query row r = TMEM lane r), warp 8 lane 0 issues TMA loads, warp 9 lane 0 issues MMAs in the
// order P0.V, Q0.K', P1.V, Q1.K' so that each group's softmax runs under the other group's MMAs.
// The running maximum is only raised when a tile exceeds it by more than 2^8 (the rescale of O is
// then rare); vertical-line columns inside low-bit tiles are knocked out by storing -inf into
// their S columns in TMEM.  Every mbarrier wait is bounded; when one expires the CTA records
// HYQ_ERR_TIMEOUT in the status word and unwinds.
#include <cuda_fp16.h>

#include "attn_common.cuh"
#include "sm100.cuh"

namespace hyq {
using namespace sm100;

constexpr int BM = 128, BN = 128, QT = 2;
constexpr int TC_THREADS = 320;
constexpr long long WAIT_LIMIT = 4000000000LL;      // SM clocks (~2 s): far beyond any legitimate wait
constexpr float RESCALE_THRESHOLD = 8.0f;           // log2 units

constexpr uint32_t SQ_OFF = 0, SQC_OFF = QT * 32768, SK_OFF = SQC_OFF + QT * 16384, SV_OFF = SK_OFF + 2 * 32768;
constexpr uint32_t TILE_SMEM = SV_OFF + 2 * 32768;                  // 229376
constexpr uint32_t TC_SMEM_BYTES = TILE_SMEM + 1024;                // + slack for 1024-byte alignment

constexpr uint32_t TM_COLS = 512;
__device__ __forceinline__ uint32_t tm_s(int q) { return q * 128; }
__device__ __forceinline__ uint32_t tm_o(int q) { return 256 + q * 128; }

constexpr uint32_t INT_MAGIC = 0x4B400000u;          // float(2^23 + 2^22): int -> float by integer add
constexpr float INT_MAGIC_F = 12582912.0f;
constexpr uint32_t KNOCKOUT_F32 = 0xFF800000u;       // -inf
constexpr uint32_t KNOCKOUT_S32 = KNOCKOUT_F32 - INT_MAGIC;   // becomes -inf after the magic add

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
    long long* timing;           // profiling builds only (HYQ_TC_TIMING): per-section cycle sums of CTA 0
};

struct TcBarriers {
    uint64_t q_full, k_full[2], k_free[2], v_full[2], v_free[2], s_full[QT], p_full[QT], o_done[QT];
};

// which key tiles a 128-row query tile visits in each pass
struct QSched {
    int live, i0, i1, nA, nB, tC0, tC1;
};

#ifdef HYQ_TC_TIMING
#define TSTAMP(var) const long long var = clock64()
#define TACC(slot, a, b) tacc[slot] += (b) - (a)
#else
#define TSTAMP(var)
#define TACC(slot, a, b)
#endif

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

// ---- softmax building blocks: one thread = one query row of 128 scores held in registers ---------
// row maximum of the raw scores of one 64-column half (integer scores are compared as integers)
template <bool INT>
__device__ __forceinline__ float half_max(const uint32_t (&raw)[BN], int h) {
    if (INT) {
        int m0 = (int)raw[h * 64], m1 = (int)raw[h * 64 + 1];
#pragma unroll
        for (int e = 2; e < 64; e += 2) {
            m0 = max(m0, (int)raw[h * 64 + e]);
            m1 = max(m1, (int)raw[h * 64 + e + 1]);
        }
        const int m = max(m0, m1);
        return (m < -(1 << 23)) ? -INFINITY : (float)m;      // knocked-out entries sit far below any score
    } else {
        float m0 = __uint_as_float(raw[h * 64]), m1 = __uint_as_float(raw[h * 64 + 1]);
#pragma unroll
        for (int e = 2; e < 64; e += 2) {
            m0 = fmaxf(m0, __uint_as_float(raw[h * 64 + e]));
            m1 = fmaxf(m1, __uint_as_float(raw[h * 64 + e + 1]));
        }
        return fmaxf(m0, m1);
    }
}

// p = 2^(raw * c + bias) for 32 columns starting at `col0`, packed to fp16 pairs; returns their fp32 sum
template <bool INT>
__device__ __forceinline__ float exp_chunk(const uint32_t (&raw)[BN], int col0, float c, float bias, uint32_t (&pk)[16]) {
    float s0 = 0.0f, s1 = 0.0f, s2 = 0.0f, s3 = 0.0f;
#pragma unroll
    for (int e = 0; e < 32; e += 4) {
        float pv[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const uint32_t rv = raw[col0 + e + u];
            const float x = INT ? __uint_as_float(rv + INT_MAGIC) : __uint_as_float(rv);
            pv[u] = ex2f(fmaf(x, c, bias));
        }
        s0 += pv[0]; s1 += pv[1]; s2 += pv[2]; s3 += pv[3];
        const __half2 h01 = __floats2half2_rn(pv[0], pv[1]), h23 = __floats2half2_rn(pv[2], pv[3]);
        pk[e >> 1] = *reinterpret_cast<const uint32_t*>(&h01);
        pk[(e >> 1) + 1] = *reinterpret_cast<const uint32_t*>(&h23);
    }
    return (s0 + s1) + (s2 + s3);
}

// one tile of the online softmax for one query row: S (TMEM) -> running (m, l) -> P (TMEM, fp16)
// returns false when a bounded wait expired
template <bool INT>
__device__ __forceinline__ bool softmax_tile(uint32_t ts, uint32_t to, float cs0, float cs1, bool first, uint64_t* o_done,
                                             uint32_t o_parity, float& m_used, float& l_run) {
    uint32_t raw[BN];
    {
        uint32_t (*r4)[32] = reinterpret_cast<uint32_t (*)[32]>(raw);
        tmem_ld32(ts, r4[0]);
        tmem_ld32(ts + 32, r4[1]);
        tmem_ld32(ts + 64, r4[2]);
        tmem_ld32(ts + 96, r4[3]);
        tmem_wait_ld();
    }
    const float f0 = half_max<INT>(raw, 0), f1 = half_max<INT>(raw, 1);
    const float mt = fmaxf(f0 == -INFINITY ? -INFINITY : f0 * cs0, f1 == -INFINITY ? -INFINITY : f1 * cs1);

    // raise the running maximum only when the tile exceeds it by the threshold
    float alpha = 1.0f;
    const bool raise = mt > m_used + RESCALE_THRESHOLD;          // also true for the first finite maximum
    if (raise) {
        alpha = ex2f(m_used - mt);                               // m_used = -inf -> 0
        l_run *= alpha;
        m_used = mt;
    }
    if (!first && __any_sync(0xffffffffu, raise)) {
        // the previous P.V of this query tile must have landed before O is rescaled
        if (!mbar_wait(o_done, o_parity, WAIT_LIMIT)) return false;
        __syncwarp();
        tc_fence_after();
#pragma unroll 1
        for (int c = 0; c < 4; ++c) {
            uint32_t o[32];
            tmem_ld32(to + c * 32, o);
            tmem_wait_ld();
#pragma unroll
            for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
            tmem_st32(to + c * 32, o);
        }
    }
    const float m_eff = (m_used == -INFINITY) ? 0.0f : m_used;
    const float b0 = INT ? fmaf(-INT_MAGIC_F, cs0, -m_eff) : -m_eff;
    const float b1 = INT ? fmaf(-INT_MAGIC_F, cs1, -m_eff) : -m_eff;
    float rs = 0.0f;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        uint32_t pk[16];
        rs += exp_chunk<INT>(raw, c * 32, (c < 2) ? cs0 : cs1, (c < 2) ? b0 : b1, pk);
        tmem_st16(ts + c * 16, pk);
    }
    l_run += rs;
    tmem_wait_st();
    return true;
}

// boundary tiles: columns outside [lo_eff, lo_eff + span] of this row are set to -inf in TMEM
__device__ __forceinline__ void mask_tile_in_tmem(uint32_t ts, int lo_eff, unsigned span, uint32_t knock) {
#pragma unroll 1
    for (int c = 0; c < 4; ++c) {
        uint32_t raw[32];
        tmem_ld32(ts + c * 32, raw);
        tmem_wait_ld();
#pragma unroll
        for (int e = 0; e < 32; ++e) raw[e] = ((unsigned)(c * 32 + e - lo_eff) <= span) ? raw[e] : knock;
        tmem_st32(ts + c * 32, raw);
    }
    tmem_wait_st();
}

template <bool LOWBIT_FP8>
__global__ void __launch_bounds__(TC_THREADS, 1)
attn_tc_kernel(const __grid_constant__ TcMaps maps, const TcParams p) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    __shared__ TcBarriers bars;
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s, cnt_b_s[QT];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int pt = gridDim.x - 1 - blockIdx.x;               // pair of query tiles; longest rows first
    const int h = blockIdx.y, b = blockIdx.z;
    const int L = p.L, W = p.window, g = p.Hq / p.Hkv;
    const int qhead = b * p.Hq + h, kvhead = b * p.Hkv + h / g;
    const int32_t* idx_row = p.vl_idx + (long)qhead * p.k;

    if (threadIdx.x == 0) {
        mbar_init(&bars.q_full, 1);
        for (int s = 0; s < 2; ++s) {
            mbar_init(&bars.k_full[s], 1);
            mbar_init(&bars.k_free[s], 1);
            mbar_init(&bars.v_full[s], 1);
            mbar_init(&bars.v_free[s], 1);
        }
        for (int q = 0; q < QT; ++q) {
            mbar_init(&bars.s_full[q], 1);
            mbar_init(&bars.p_full[q], 128);
            mbar_init(&bars.o_done[q], 1);
        }
        fence_mbar_init();
        abort_s = 0;
    }
    if (threadIdx.x < QT) {
        const int i1 = min(pt * QT * BM + threadIdx.x * BM + BM - 1, L - 1);
        cnt_b_s[threadIdx.x] = (p.k > 0 && i1 - W >= 0) ? count_le(idx_row, p.k, i1 - W) : 0;
    }
    if (warp == 8) {
        tmem_alloc(&tmem_base_s, TM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_base_s;

    // per query tile: nA low-bit tiles, nB gathered vertical-line tiles, window tiles tC0..tC1
    QSched qs[QT];
#pragma unroll
    for (int q = 0; q < QT; ++q) {
        QSched& s = qs[q];
        s.i0 = (pt * QT + q) * BM;
        s.live = s.i0 < L;
        s.i1 = min(s.i0 + BM - 1, L - 1);
        s.nA = (s.live && s.i1 - W >= 0) ? (s.i1 - W) / BN + 1 : 0;
        s.nB = s.live ? (cnt_b_s[q] + BN - 1) / BN : 0;
        s.tC0 = max(0, s.i0 - W + 1) / BN;
        s.tC1 = (s.live && W > 0) ? s.i1 / BN : -1;
    }
    // the CTA walks the union of both lists (tile 1 holds the later rows, so its lists are the longer ones)
    const int nA = max(qs[0].nA, qs[1].nA), nB = max(qs[0].nB, qs[1].nB);
    const int tC0 = qs[0].tC0, tC1 = max(qs[0].tC1, qs[1].tC1);
    const int nC = (W > 0) ? tC1 - tC0 + 1 : 0;
    const int T = nA + nB + nC;
    auto active = [&](int q, int t) -> bool {
        const QSched& s = qs[q];
        if (!s.live) return false;
        if (t < nA) return t < s.nA;
        if (t < nA + nB) return t - nA < s.nB;
        const int tile = tC0 + t - nA - nB;
        return tile >= s.tC0 && tile <= s.tC1;
    };

    volatile int* abort_flag = &abort_s;
    auto fail = [&]() {
        *abort_flag = 1;
        if (p.status) atomicExch(p.status, HYQ_ERR_TIMEOUT);
    };

    if (warp == 8) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            prefetch_tmap(&maps.q);
            prefetch_tmap(&maps.k);
            prefetch_tmap(&maps.kc);
            prefetch_tmap(&maps.vh16);
            uint32_t qbytes = 0;
            for (int q = 0; q < QT; ++q)
                if (qs[q].live) qbytes += 32768 + (nA > 0 ? 16384 : 0);
            mbar_arrive_expect_tx(&bars.q_full, qbytes);
            for (int q = 0; q < QT; ++q) {
                if (!qs[q].live) continue;
                tma_load_3d(smem + SQ_OFF + q * 32768, &maps.q, &bars.q_full, 0, qs[q].i0, qhead);
                tma_load_3d(smem + SQ_OFF + q * 32768 + 16384, &maps.q, &bars.q_full, 64, qs[q].i0, qhead);
                if (nA > 0) tma_load_3d(smem + SQC_OFF + q * 16384, &maps.qc, &bars.q_full, 0, qs[q].i0, qhead);
            }
            for (int t = 0; t < T && !*abort_flag; ++t) {
                const int s = t & 1, u = t >> 1;
                unsigned char* sk = smem + SK_OFF + s * 32768;
                unsigned char* sv = smem + SV_OFF + s * 32768;
                const bool lowbit = t < nA, vl = !lowbit && t < nA + nB;
                const int row = lowbit ? t * BN : (vl ? (t - nA) * BN : (tC0 + t - nA - nB) * BN);
                const int hd = vl ? qhead : kvhead;
                if (u > 0 && !mbar_wait(&bars.k_free[s], (u - 1) & 1, WAIT_LIMIT)) { fail(); break; }
                if (lowbit) {
                    mbar_arrive_expect_tx(&bars.k_full[s], 16384);
                    tma_load_3d(sk, &maps.kc, &bars.k_full[s], 0, row, hd);
                } else {
                    const CUtensorMap* m = vl ? &maps.kvl : &maps.k;
                    mbar_arrive_expect_tx(&bars.k_full[s], 32768);
                    tma_load_3d(sk, m, &bars.k_full[s], 0, row, hd);
                    tma_load_3d(sk + 16384, m, &bars.k_full[s], 64, row, hd);
                }
                if (u > 0 && !mbar_wait(&bars.v_free[s], (u - 1) & 1, WAIT_LIMIT)) { fail(); break; }
                {
                    const CUtensorMap* m = lowbit ? &maps.vh16 : (vl ? &maps.vvl : &maps.v16);
                    mbar_arrive_expect_tx(&bars.v_full[s], 32768);
                    tma_load_3d(sv, m, &bars.v_full[s], 0, row, hd);
                    tma_load_3d(sv + 16384, m, &bars.v_full[s], 64, row, hd);
                }
            }
        }
    } else if (warp == 9) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t idesc_lq = LOWBIT_FP8 ? make_idesc(ACC_F32, FMT_E4M3, FMT_E4M3, 0, 0, BM, BN)
                                                   : make_idesc(ACC_S32, FMT_S8, FMT_S8, 0, 0, BM, BN);
            const uint32_t idesc_qk = make_idesc(ACC_F32, FMT_BF16, FMT_BF16, 0, 0, BM, BN);
            const uint32_t idesc_pv = make_idesc(ACC_F32, FMT_F16, FMT_F16, 0, 1, BM, HYQ_D);
            int n_pv[QT] = {0, 0};
            bool ok = mbar_wait(&bars.q_full, 0, WAIT_LIMIT);
            auto wait_k = [&](int t) { return mbar_wait(&bars.k_full[t & 1], (t >> 1) & 1, WAIT_LIMIT); };
            auto issue_qk = [&](int q, int t) {
                if (!active(q, t)) return;
                const uint32_t sk = smem_u32(smem + SK_OFF + (t & 1) * 32768);
                const uint32_t d = tmem + tm_s(q);
                if (t < nA) {
                    const uint32_t sqc = smem_u32(smem + SQC_OFF + q * 16384);
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk) {
                        const uint64_t da = make_smem_desc(sqc + kk * 32, 0, 1024), db = make_smem_desc(sk + kk * 32, 0, 1024);
                        if (LOWBIT_FP8) umma_ss_f8f6f4(d, da, db, idesc_lq, kk > 0);
                        else umma_ss_i8(d, da, db, idesc_lq, kk > 0);
                    }
                } else {
                    const uint32_t sq = smem_u32(smem + SQ_OFF + q * 32768);
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk) {
                        const uint32_t off = (kk >> 2) * 16384 + (kk & 3) * 32;
                        umma_ss_f16(d, make_smem_desc(sq + off, 0, 1024), make_smem_desc(sk + off, 0, 1024), idesc_qk, kk > 0);
                    }
                }
                umma_commit(&bars.s_full[q]);
            };
            auto issue_pv = [&](int q, int t) -> bool {
                if (!active(q, t)) return true;
                if (!mbar_wait(&bars.p_full[q], n_pv[q] & 1, WAIT_LIMIT)) return false;
                tc_fence_after();
                const uint32_t sv = smem_u32(smem + SV_OFF + (t & 1) * 32768);
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)
                    umma_ts_f16(tmem + tm_o(q), tmem + tm_s(q) + kk * 8, make_smem_desc(sv + kk * 2048, 16384, 1024), idesc_pv,
                                (n_pv[q] > 0 || kk > 0));
                umma_commit(&bars.o_done[q]);
                ++n_pv[q];
                return true;
            };
            if (ok && T > 0) {
                ok = wait_k(0);
                if (ok) {
                    tc_fence_after();
                    issue_qk(0, 0);
                    issue_qk(1, 0);
                    umma_commit(&bars.k_free[0]);
                }
            }
            for (int t = 0; t < T && ok && !*abort_flag; ++t) {
                ok = mbar_wait(&bars.v_full[t & 1], (t >> 1) & 1, WAIT_LIMIT);
                if (!ok) break;
                ok = issue_pv(0, t);
                if (!ok) break;
                if (t + 1 < T) {
                    ok = wait_k(t + 1);
                    if (!ok) break;
                    tc_fence_after();
                    issue_qk(0, t + 1);
                }
                ok = issue_pv(1, t);
                if (!ok) break;
                umma_commit(&bars.v_free[t & 1]);
                if (t + 1 < T) {
                    issue_qk(1, t + 1);
                    umma_commit(&bars.k_free[(t + 1) & 1]);
                }
            }
            if (!ok) fail();
        }
    } else {
        // ------------------------------------------------------------------ softmax groups
        const int q = warp >> 2;
        const QSched sq = qs[q];
        const int r = threadIdx.x & 127;                // query row inside the tile = TMEM lane
        const int i = sq.i0 + r;
        const bool row_live = i < L;
        const bool ragged = sq.i0 + BM > L;
        const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t ts = tmem + tm_s(q) + lane_addr, to = tmem + tm_o(q) + lane_addr;
        const float q_scale = row_live ? __ldg(p.q_scales + (long)qhead * p.nb + i / HYQ_BLOCK_TOKENS) : 0.0f;
        const int cnt_r = (sq.nB > 0 && row_live && i - W >= 0) ? count_le(idx_row, p.k, i - W) : 0;
        const uint32_t* bits_row = p.vl_bits + (long)qhead * p.mask_words;
        float m_used = -INFINITY, l_run = 0.0f;
        int n_act = 0;
        bool ok = true;

        // scales and vertical-line bitmask words of a low-bit tile, fetched one tile ahead of their use
        float nk0 = 0.0f, nk1 = 0.0f;
        uint32_t nvl[4] = {0u, 0u, 0u, 0u};
        auto prefetch_tile = [&](int t) {
            if (t >= nA) return;
            nk0 = __ldg(p.k_scales + (long)kvhead * p.nb + min(2 * t, p.nb - 1));
            nk1 = __ldg(p.k_scales + (long)kvhead * p.nb + min(2 * t + 1, p.nb - 1));
#pragma unroll
            for (int w = 0; w < 4; ++w) nvl[w] = (t * 4 + w < p.mask_words) ? __ldg(bits_row + t * 4 + w) : 0u;
        };
        prefetch_tile(0);
#ifdef HYQ_TC_TIMING
        long long tacc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
#endif

        for (int t = 0; t < T; ++t) {
            const float k0 = nk0, k1 = nk1;
            uint32_t vlw[4] = {nvl[0], nvl[1], nvl[2], nvl[3]};
            prefetch_tile(t + 1);
            if (!active(q, t)) continue;
            // ---- per-tile column bounds and scales
            int lo = 0, hi = -1;
            bool need_range;
            float cs0, cs1;
            const bool lowbit = t < nA;
            if (lowbit) {
                const int j0 = t * BN;
                hi = row_live ? min(i - W - j0, BN - 1) : -1;
                need_range = (j0 + BN - 1 > sq.i0 - W) || ragged;
                // a zero scale (all-zero tile) still has to let -inf pass through the multiply
                cs0 = fmaxf(q_scale * k0 * p.scale_log2, 1e-37f);
                cs1 = fmaxf(q_scale * k1 * p.scale_log2, 1e-37f);
            } else if (t < nA + nB) {
                const int c0 = (t - nA) * BN;
                hi = min(cnt_r - c0 - 1, BN - 1);
                need_range = true;
                cs0 = cs1 = p.scale_log2;
                vlw[0] = vlw[1] = vlw[2] = vlw[3] = 0u;
            } else {
                const int j0 = (tC0 + t - nA - nB) * BN;
                lo = max(0, i - W + 1 - j0);
                hi = row_live ? min(i - j0, BN - 1) : -1;
                need_range = (j0 + BN - 1 > sq.i0) || (j0 <= sq.i1 - W) || ragged;
                cs0 = cs1 = p.scale_log2;
                vlw[0] = vlw[1] = vlw[2] = vlw[3] = 0u;
            }
            const int lo_eff = (hi >= lo) ? lo : 4096;
            const unsigned span = (hi >= lo) ? (unsigned)(hi - lo) : 0u;
            const bool int_scores = lowbit && !LOWBIT_FP8;

            TSTAMP(c0_);
            if (!mbar_wait(&bars.s_full[q], n_act & 1, WAIT_LIMIT)) { ok = false; break; }
            __syncwarp();
            tc_fence_after();
            TSTAMP(c1_);

            const uint32_t knock = int_scores ? KNOCKOUT_S32 : KNOCKOUT_F32;
            // ---- boundary tiles: causal / window / validity limits of this row, applied in TMEM
            if (need_range) mask_tile_in_tmem(ts, lo_eff, span, knock);
            // ---- vertical-line keys inside a low-bit tile: their S columns become -inf
            if ((vlw[0] | vlw[1] | vlw[2] | vlw[3]) != 0u) {
#pragma unroll
                for (int w = 0; w < 4; ++w) {
                    uint32_t bits = vlw[w];
                    while (bits) {
                        const int c = __ffs(bits) - 1;
                        bits &= bits - 1;
                        tmem_st1(ts + w * 32 + c, knock);
                    }
                }
                tmem_wait_st();
            }
            TSTAMP(c2_);
            if (int_scores) ok = softmax_tile<true>(ts, to, cs0, cs1, n_act == 0, &bars.o_done[q], (n_act - 1) & 1, m_used, l_run);
            else ok = softmax_tile<false>(ts, to, cs0, cs1, n_act == 0, &bars.o_done[q], (n_act - 1) & 1, m_used, l_run);
            if (!ok) break;
            TSTAMP(c3_);
            tc_fence_before();
            mbar_arrive(&bars.p_full[q]);
            TSTAMP(c4_);
            TACC(0, c0_, c1_); TACC(1, c1_, c2_); TACC(2, c2_, c3_); TACC(3, c3_, c4_);
#ifdef HYQ_TC_TIMING
            tacc[4] += 1;
#endif
            ++n_act;
        }
#ifdef HYQ_TC_TIMING
        if (p.timing && blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0 && (threadIdx.x & 127) == 0)
            for (int e = 0; e < 5; ++e) p.timing[q * 8 + e] = tacc[e];
#endif

        // ---- epilogue: O / l
        if (ok && n_act > 0) ok = mbar_wait(&bars.o_done[q], (n_act - 1) & 1, WAIT_LIMIT);
        __syncwarp();
        if (ok && n_act > 0) {
            tc_fence_after();
            const float inv = (l_run > 0.0f) ? 1.0f / l_run : 0.0f;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t o[32];
                tmem_ld32(to + c * 32, o);
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
            if (p.lse && row_live) p.lse[(long)qhead * L + i] = (m_used + log2f(l_run)) * 0.6931471805599453f;
        } else if (!ok) {
            fail();
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 8) {
        __syncwarp();
        tmem_dealloc(tmem, TM_COLS);
    }
}

// ---------------------------------------------------------------------------------------------
#ifdef HYQ_TC_TIMING
static __device__ long long g_timing[16];
extern "C" int hyq_debug_read_timing(long long* host16) {
    return cudaMemcpyFromSymbol(host16, g_timing, sizeof(long long) * 16) == cudaSuccess ? 0 : 5;
}
#endif

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
    p.timing = nullptr;
#ifdef HYQ_TC_TIMING
    cudaGetSymbolAddress(reinterpret_cast<void**>(&p.timing), g_timing);
#endif

    auto kern = int4 ? attn_tc_kernel<true> : attn_tc_kernel<false>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)TC_SMEM_BYTES) != cudaSuccess)
        return HYQ_ERR_CUDA;
    const dim3 grid((a.L + QT * BM - 1) / (QT * BM), a.Hq, a.B);
    if (a.ev_kernel_start && cudaEventRecord(static_cast<cudaEvent_t>(a.ev_kernel_start), st) != cudaSuccess) return HYQ_ERR_CUDA;
    kern<<<grid, TC_THREADS, TC_SMEM_BYTES, st>>>(maps, p);
    if (launch_status() != HYQ_OK) return HYQ_ERR_CUDA;
    if (a.ev_kernel_stop && cudaEventRecord(static_cast<cudaEvent_t>(a.ev_kernel_stop), st) != cudaSuccess) return HYQ_ERR_CUDA;
    return HYQ_OK;
}

}  // namespace hyq
