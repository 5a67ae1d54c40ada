// Fused hybrid-precision causal attention (Eq. 6-7; Algorithm 2, Stage 3) on the 5th-generation
// tensor cores: TMA -> shared memory -> tcgen05.mma -> TMEM, one online softmax over three passes.
//
// One CTA owns 256 query rows (two 128-row tiles) of one (b, query head) and walks key tiles of 64
// (one quantization block, so one K scale per tile):
//   pass A  low-bit keys   j <= i - W, j not vertical   S = Qc.Kc^T  (kind::i8, or kind::f8f6f4 on
//                                                       INT4 codes widened to e4m3), V^ in fp16
//   pass B  vertical keys  gathered per query head, ascending, idx <= i - W   S = Q.Kvl^T (bf16)
//   pass C  window keys    i - W < j <= i                                     S = Q.K^T   (bf16)
// All passes feed one running (m, l) per row and one fp32 O accumulator per query tile in TMEM.
// S is double-buffered per query tile (4 x 64 TMEM columns), so Q.K^T of the next tile is done
// before the softmax of the current one ends; P goes back to TMEM as fp16 over the S columns it
// was computed from and is the A operand of the P.V MMA (fp16 x fp16).  The K tile and the V tile of
// a walk position share one stage of a 4-stage ring (one "full" and one "free" barrier per stage) and
// are used by both query tiles.
//
// Warp roles (384 threads): warp 0 lane 0 issues the TMA loads, warps 1 and 2 (lane 0) issue the
// MMAs of query tile 0 and 1 (four tiles per trip with compile-time ring positions in the steady
// state of the low-bit pass), warp 3 idles, warps 4-11 are the softmax warps: four per query tile,
// one thread per query row (row r = TMEM lane r of every score tile; the thread holds the 64 scores
// of its row in two register halves), so a row's reference maximum needs no agreement between
// threads.  The exponentials are taken against that reference, which is only raised when
// a tile exceeds it by more than 2^14 (the rescale of O is then rare); integer scores become floats
// by a magic-number add.  The vertical-line keys inside a low-bit tile are taken out of pass A before the
// softmax sees the scores: with e4m3 codes by a fifth MMA step per tile, S += ones . mask^T in e5m2 (the one
// 8-bit format with an infinity), whose 64 x 32 operand - -inf in element 0 of a vertical key's row - is copied
// in with the K codes; with int8 codes (no infinity) by the softmax warps, which store -inf over those columns
// of S before they read the tile.  The attention call launches the kernel twice: the first launch takes most low-bit
// tiles without looking for their maximum and checks the tiles' row sums instead, the second redoes the CTAs (normally
// none) in which that check failed - see the comment at attn_tc_kernel.  Every mbarrier wait is bounded; when one expires the CTA records
// HYQ_ERR_TIMEOUT in the status word, waits (bounded) for its own copies and MMAs in flight and unwinds.
#include <cuda_fp16.h>

#include <type_traits>

#include "attn_common.cuh"
#include "sm100.cuh"

// This file is compiled twice: as it stands (64-token quantization blocks, the size every workload uses) and,
// through attn_tc_bt.cu with HYQ_TC_VARIANT_BT = 1, a second time into namespace hyq::tcbt with the block size a
// run-time parameter (32 or 128 tokens).  The kernel's loop is sensitive to every live register - compiling the
// parameter in, even behind a compile-time-false branch, cost the 64-token path 5 % - so the default translation
// unit carries nothing of it.  With 32-token blocks the two column halves of a tile have separate K scales: the
// softmax thread then applies each half's own factor.
#ifndef HYQ_TC_VARIANT_BT
#define HYQ_TC_VARIANT_BT 0
#endif
namespace hyq {
#if HYQ_TC_VARIANT_BT
namespace tcbt {
#endif
using namespace sm100;

constexpr int BM = 128, QT = 2;
constexpr int RING_BYTES = 65536;                   // shared memory of the K ring and of the V ring
constexpr long long WAIT_LIMIT_DEFAULT = 4000000000LL;   // SM clocks (~2 s): far beyond any legitimate wait

constexpr uint32_t Q_TILE_BYTES = BM * HYQ_D * 2, QC_TILE_BYTES = BM * HYQ_D;        // 32768, 16384
constexpr uint32_t SQ_OFF = 0, SQC_OFF = QT * Q_TILE_BYTES, SK_OFF = SQC_OFF + QT * QC_TILE_BYTES;
constexpr uint32_t SV_OFF = SK_OFF + RING_BYTES;
constexpr uint32_t TILE_SMEM = SV_OFF + RING_BYTES;                 // 229376
constexpr int MAX_STAGES = 4;
// In the low-bit pass a K ring slot holds 8 KB of codes; behind them sit the vertical-line operand of the tile
// (64 keys x 32 e5m2 elements, copied in with the codes) and this slot's copy of the constant 128 x 32 operand whose
// element 0 of every row is one.
constexpr uint32_t VLT_OFF = 8192, ONES_OFF = 10240, ONES_BYTES = 4096;

// geometry that follows from the keys per tile (64: 4-stage ring, two S buffers per query tile)
template <int TBN> struct Geo {
    static constexpr int BN = TBN;
    static constexpr int NBUF = 128 / TBN;                              // S buffers per query tile (128 TMEM columns)
    static constexpr uint32_t STAGE_BYTES = TBN * HYQ_D * 2;            // one bf16 / fp16 tile
    static constexpr uint32_t KC_TILE_BYTES = TBN * HYQ_D;              // one tile of 8-bit codes
    static constexpr int NST = RING_BYTES / STAGE_BYTES;                // ring depth
    static constexpr int NSC = TBN / 64;                                // K scales (quantization blocks) per tile
    static constexpr int NVW = TBN / 32;                                // vertical-line bitmask words per tile
};
constexpr uint32_t TC_SMEM_BYTES = TILE_SMEM + 1024;                // + slack for 1024-byte alignment

constexpr uint32_t TM_COLS = 512;
__device__ __forceinline__ uint32_t tm_s(int q) { return q * 128; }      // + buffer * BN
__device__ __forceinline__ uint32_t tm_o(int q) { return 256 + q * 128; }

constexpr uint32_t INT_MAGIC = 0x4B400000u;          // float(2^23 + 2^22): int -> float by integer add
constexpr float INT_MAGIC_F = 12582912.0f;
constexpr uint32_t KNOCKOUT_F32 = 0xFF800000u;       // -inf
constexpr uint32_t KNOCKOUT_S32 = KNOCKOUT_F32 - INT_MAGIC;   // becomes -inf after the magic add

// CTAs whose work was done a second time by the exact kernel (read and reset by the test hook)
__device__ unsigned long long g_tc_restarts = 0ull;

struct TcMaps {
    CUtensorMap q, k, qc, kc, v16, vh16, kvl, vvl;
};

struct TcParams {
    int B, Hq, Hkv, L, window, k, nb, mask_words;
#if HYQ_TC_VARIANT_BT
    int bt_shift;                // log2(tokens per quantization block): 5 or 7
#endif
    int Lq, nbq;                 // query rows (end-aligned with the L keys: row i sits at position L - Lq + i), their blocks
    int fixed_tail;              // window form: the last `window` keys for every row instead of each row's own
    int splits;                  // CTAs per pair of query tiles, each on a slice of the walk (short query blocks)
    float* part_o;               // splits > 1: unnormalised partial outputs [splits][B*Hq][Lq][D] ...
    float* part_ml;              // ... and (reference maximum in log2 units, row sum) [splits][B*Hq][Lq][2]
    int out_fp32;
    float scale_log2;            // softmax_scale * log2(e)
    const float* q_scales;
    const float* k_scales;
    const int32_t* vl_idx;
    const uint32_t* vl_bits;
    uint32_t* redo;              // [0]: number of CTAs of the optimistic kernel that gave up, [1 + 3 i ...]: their block indices
    int grid_x;                  // blockIdx.x range of the optimistic kernel (pairs of query tiles x slices)
    const uint8_t* vl_tiles;     // FP8 / INT4 scores: the vertical-line operand tiles [B*Hq][mask_words/2][2048] (null: none)
    void* out;
    float* lse;
    int32_t* status;
    long long wait_limit;        // SM clocks a single barrier wait may take
    int drop_load;               // test hook: walk position whose K/V load the producer announces but never issues (-1: none)
};

struct TcBarriers {
    uint64_t q_full, kv_full[MAX_STAGES], kv_free[MAX_STAGES];   // ring stage = K tile and V tile of one walk position
    uint64_t s_full[QT][2], p_full[QT][2], o_done[QT][2], drain[QT];
};

// which key tiles a 128-row query tile visits in each pass (i0, i1: first and last row of the tile in the query
// block; the tile lists follow from their positions among the keys)
struct QSched {
    int live, i0, i1, nA, nB, tC0, tC1;
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

// the tile walk of one CTA: union of both query tiles' lists
struct Walk {
    int nA, nB, tC0, nC, T;
    int t0, t1;                 // the positions [t0, t1) this CTA works on (all of [0, T) unless the keys are split)
};

// own tile ranges of one query tile inside the CTA's walk: [0, a_end) low-bit, [b_beg, b_end) vertical, [c_beg, c_end) window
struct OwnTiles {
    int a_end, b_beg, b_end, c_beg, c_end;
    __device__ __forceinline__ bool has(int t) const { return t < a_end || (t >= b_beg && t < b_end) || (t >= c_beg && t < c_end); }
};
// number of own tiles at walk positions below t
__device__ __forceinline__ int own_before(const OwnTiles& o, int t) {
    return min(t, o.a_end) + min(max(t - o.b_beg, 0), o.b_end - o.b_beg) + min(max(t - o.c_beg, 0), o.c_end - o.c_beg);
}
__device__ __forceinline__ OwnTiles own_tiles(const QSched& s, const Walk& w) {
    OwnTiles o;
    o.a_end = s.live ? s.nA : 0;
    o.b_beg = w.nA;
    o.b_end = s.live ? w.nA + s.nB : w.nA;
    o.c_beg = w.nA + w.nB + (s.tC0 - w.tC0);
    o.c_end = (s.live && s.tC1 >= s.tC0) ? w.nA + w.nB + (s.tC1 - w.tC0) + 1 : o.c_beg;
    return o;
}

// MMA issue for one query tile (one thread): S = Q.K^T runs NBUF tiles ahead of the softmax, O += P.V behind it.
// The loop body is kept to waits, MMAs and commits: ring positions, parities and descriptors advance incrementally.
template <bool LOWBIT_FP8, int TBN>
__device__ __forceinline__ bool mma_issuer(int q, const QSched& sq, const Walk& w, TcBarriers& bars, unsigned char* smem,
                                           uint32_t tmem, volatile int* abort_flag, long long limit, bool vl_mma) {
    using G = Geo<TBN>;
    constexpr int BN = TBN, NST = G::NST, NBUF = G::NBUF;
    constexpr uint32_t STAGE16 = G::STAGE_BYTES >> 4;                  // descriptor address units per ring stage
    const uint32_t idesc_lq = LOWBIT_FP8 ? make_idesc(ACC_F32, FMT_E4M3, FMT_E4M3, 0, 0, BM, BN)
                                         : make_idesc(ACC_S32, FMT_S8, FMT_S8, 0, 0, BM, BN);
    const uint32_t idesc_qk = make_idesc(ACC_F32, FMT_BF16, FMT_BF16, 0, 0, BM, BN);
    const uint32_t idesc_pv = make_idesc(ACC_F32, FMT_F16, FMT_F16, 0, 1, BM, HYQ_D);
    const uint64_t dq = make_smem_desc(smem_u32(smem + SQ_OFF + q * Q_TILE_BYTES), 0, 1024);
    const uint64_t dqc = make_smem_desc(smem_u32(smem + SQC_OFF + q * QC_TILE_BYTES), 0, 1024);
    const uint64_t dk0 = make_smem_desc(smem_u32(smem + SK_OFF), 0, 1024);
    const uint64_t dv0 = make_smem_desc(smem_u32(smem + SV_OFF), G::STAGE_BYTES / 2, 1024);
    // S += ones . mask^T: -inf on the columns of vertical-line keys, +0 elsewhere (e5m2 has an infinity, e4m3 has not)
    const uint32_t idesc_vl = make_idesc(ACC_F32, FMT_E5M2, FMT_E5M2, 0, 0, BM, BN);
    const uint64_t dones0 = make_smem_desc_plain(smem_u32(smem + SK_OFF + ONES_OFF), BM * 16, 128);
    const uint64_t dvlt0 = make_smem_desc_plain(smem_u32(smem + SK_OFF + VLT_OFF), BN * 16, 128);
    const uint32_t ts0 = tmem + tm_s(q), to = tmem + tm_o(q);
    const OwnTiles own = own_tiles(sq, w);
    const int nA = w.nA;
    if (!mbar_wait(&bars.q_full, 0, limit)) return false;

    // Q.K^T cursor
    int tq = w.t0, kst = 0;
    uint32_t kpar = 0, n_qk = 0;
    const int T1 = w.t1;
    // (k_ready: the stage of position tq is already known to have landed)
    auto qk = [&](bool k_ready) -> bool {
        if (!k_ready && !mbar_wait(&bars.kv_full[kst], kpar, limit)) return false;
        if (own.has(tq)) {
            tc_fence_after();
            const uint64_t dk = dk0 + (uint64_t)(kst * STAGE16);
            const uint32_t buf = n_qk % NBUF;
            const uint32_t d = ts0 + buf * BN;
            if (tq < nA) {
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) {
                    if (LOWBIT_FP8) umma_ss_f8f6f4(d, dqc + kk * 2, dk + kk * 2, idesc_lq, kk > 0);
                    else umma_ss_i8(d, dqc + kk * 2, dk + kk * 2, idesc_lq, kk > 0);
                }
                if (LOWBIT_FP8 && vl_mma) umma_ss_f8f6f4(d, dones0 + (uint64_t)(kst * STAGE16), dvlt0 + (uint64_t)(kst * STAGE16), idesc_vl, 1u);
            } else {
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)
                    umma_ss_f16(d, dq + ((kk >> 2) * (Q_TILE_BYTES / 32) + (kk & 3) * 2),
                                dk + ((kk >> 2) * (G::STAGE_BYTES / 32) + (kk & 3) * 2), idesc_qk, kk > 0);
            }
            umma_commit(&bars.s_full[q][buf]);
            ++n_qk;
        }
        ++tq;
        if (++kst == NST) { kst = 0; kpar ^= 1u; }
        return true;
    };
    // P.V cursor
    int vst = 0;
    uint32_t n_pv = 0;
    for (int t = 0; t < NBUF && tq < T1; ++t)
        if (!qk(false)) return false;
    // Steady state of the low-bit pass, four walk positions per trip: this thread's pace is set by the dependent
    // instructions it executes per tile, so ring stages, S buffers, barrier addresses and descriptors are compile-time
    // offsets here and the parities change once per trip.  Taken only where the cursors are in phase (V stage 0,
    // K stage 2, even tile counts) and all eight tiles involved are low-bit tiles of this query tile.
    constexpr bool FAST = (NST == 4 && NBUF == 2);
    const uint32_t a_bars = smem_u32(&bars);
    const int fast_end = min(own.a_end, T1) - 5;
    for (int t = w.t0; t < T1; ++t) {
        if (FAST && t < fast_end && vst == 0 && kst == 2 && n_pv > 0 && ((n_pv | n_qk) & 1u) == 0 && tq == t + 2) {
            const uint32_t pp = (n_pv >> 1) & 1u;
            bool ok = true;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int ks = (2 + i) & 3, bf = i & 1;
                const uint32_t a_p = a_bars + (uint32_t)offsetof(TcBarriers, p_full) + (q * 2 + bf) * 8;
                const uint32_t a_kf = a_bars + (uint32_t)offsetof(TcBarriers, kv_full) + ks * 8;
                const uint32_t ppi = i < 2 ? pp : pp ^ 1u, kpi = i < 2 ? kpar : kpar ^ 1u;
                const uint32_t done = mbar_test_wait2_a(a_p, ppi, a_kf, kpi);
                if (!(done & 1u) && !mbar_wait_a(a_p, ppi, limit)) { ok = false; break; }
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < BN / 16; ++kk)
                    umma_ts_f16(to, ts0 + bf * BN + kk * 8, dv0 + (uint64_t)(i * STAGE16 + kk * 128), idesc_pv, 1u);
                umma_commit_a(a_bars + (uint32_t)offsetof(TcBarriers, o_done) + (q * 2 + bf) * 8);
                umma_commit_a(a_bars + (uint32_t)offsetof(TcBarriers, kv_free) + i * 8);
                if (!(done & 2u) && !mbar_wait_a(a_kf, kpi, limit)) { ok = false; break; }
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) {
                    if (LOWBIT_FP8) umma_ss_f8f6f4(ts0 + bf * BN, dqc + kk * 2, dk0 + (uint64_t)(ks * STAGE16 + kk * 2), idesc_lq, kk > 0);
                    else umma_ss_i8(ts0 + bf * BN, dqc + kk * 2, dk0 + (uint64_t)(ks * STAGE16 + kk * 2), idesc_lq, kk > 0);
                }
                if (LOWBIT_FP8 && vl_mma) umma_ss_f8f6f4(ts0 + bf * BN, dones0 + (uint64_t)(ks * STAGE16), dvlt0 + (uint64_t)(ks * STAGE16), idesc_vl, 1u);
                umma_commit_a(a_bars + (uint32_t)offsetof(TcBarriers, s_full) + (q * 2 + bf) * 8);
            }
            if (!ok) return false;
            n_pv += 4; n_qk += 4; tq += 4; kpar ^= 1u; t += 3;
            if (*abort_flag) return true;
            continue;
        }
        // (the V tile of position t came in on the same barrier as its K tile, which Q.K^T waited for)
        bool k_ready = false;
        if (own.has(t)) {
            const uint32_t buf = n_pv % NBUF;
            // P of this tile, and in the same round trip the ring stage of the Q.K^T that follows
            const uint32_t done = mbar_test_wait2(&bars.p_full[q][buf], (n_pv / NBUF) & 1u, &bars.kv_full[kst], kpar);
            k_ready = (done & 2u) != 0u && tq < T1;
            if (!(done & 1u) && !mbar_wait(&bars.p_full[q][buf], (n_pv / NBUF) & 1u, limit)) return false;
            tc_fence_after();
            const uint64_t dv = dv0 + (uint64_t)(vst * STAGE16);
            const uint32_t pa = ts0 + buf * BN;
#pragma unroll
            for (int kk = 0; kk < BN / 16; ++kk) umma_ts_f16(to, pa + kk * 8, dv + kk * 128, idesc_pv, (n_pv > 0 || kk > 0));
            umma_commit(&bars.o_done[q][n_pv & 1u]);  // P.V number n of this query tile -> barrier n & 1
            ++n_pv;
            umma_commit(&bars.kv_free[vst]);        // one arrival per issuer; the ring stage is free after both
        } else {
            mbar_arrive(&bars.kv_free[vst]);        // nothing of this query tile reads the stage
        }
        if (++vst == NST) vst = 0;
        if (tq < T1 && !qk(k_ready)) return false;
        if ((t & 15) == 15 && *abort_flag) return true;
    }
    return true;
}

// TMA producer (one thread): the two query tiles once, then the K ring and the V ring along the CTA's walk
template <int TBN>
__device__ __forceinline__ bool tma_producer(const TcMaps& maps, const QSched& qs0, const QSched& qs1, const Walk& w, int qhead,
                                             int kvhead, TcBarriers& bars, unsigned char* smem, volatile int* abort_flag,
                                             long long limit, int drop_load, const uint8_t* vl_tiles, bool settle) {
    using G = Geo<TBN>;
    constexpr int BN = TBN, NST = G::NST;
    prefetch_tmap(&maps.q);
    prefetch_tmap(&maps.k);
    prefetch_tmap(&maps.kc);
    prefetch_tmap(&maps.vh16);
    const int live[QT] = {qs0.live, qs1.live}, qi0[QT] = {qs0.i0, qs1.i0};
    uint32_t qbytes = 0;
    for (int q = 0; q < QT; ++q)
        if (live[q]) qbytes += Q_TILE_BYTES + (w.nA > 0 ? QC_TILE_BYTES : 0);
    mbar_arrive_expect_tx(&bars.q_full, qbytes);
    for (int q = 0; q < QT; ++q) {
        if (!live[q]) continue;
        tma_load_3d(smem + SQ_OFF + q * Q_TILE_BYTES, &maps.q, &bars.q_full, 0, qi0[q], qhead);
        tma_load_3d(smem + SQ_OFF + q * Q_TILE_BYTES + Q_TILE_BYTES / 2, &maps.q, &bars.q_full, 64, qi0[q], qhead);
        if (w.nA > 0) tma_load_3d(smem + SQC_OFF + q * QC_TILE_BYTES, &maps.qc, &bars.q_full, 0, qi0[q], qhead);
    }
    bool ok = true;
    int t = w.t0;
    for (; t < w.t1 && !*abort_flag; ++t) {
        const int st = (t - w.t0) % NST, use = (t - w.t0) / NST;
        unsigned char* sk = smem + SK_OFF + st * G::STAGE_BYTES;
        unsigned char* sv = smem + SV_OFF + st * G::STAGE_BYTES;
        const bool lowbit = t < w.nA, vl = !lowbit && t < w.nA + w.nB;
        const int row = lowbit ? t * BN : (vl ? (t - w.nA) * BN : (w.tC0 + t - w.nA - w.nB) * BN);
        const int hd = vl ? qhead : kvhead;
        if (use > 0 && !mbar_wait_sleepy(&bars.kv_free[st], (use - 1) & 1, limit)) { ok = false; break; }
        if (lowbit) {
            mbar_arrive_expect_tx(&bars.kv_full[st], G::KC_TILE_BYTES + G::STAGE_BYTES + (vl_tiles ? VL_TILE_BYTES : 0));
            if (t == drop_load) continue;                // test hook: the announced bytes never arrive
            tma_load_3d(sk, &maps.kc, &bars.kv_full[st], 0, row, hd);
            if (vl_tiles) bulk_load_1d(sk + VLT_OFF, vl_tiles + (long)t * VL_TILE_BYTES, VL_TILE_BYTES, &bars.kv_full[st]);
        } else {
            const CUtensorMap* m = vl ? &maps.kvl : &maps.k;
            mbar_arrive_expect_tx(&bars.kv_full[st], 2 * G::STAGE_BYTES);
            if (t == drop_load) continue;
            tma_load_3d(sk, m, &bars.kv_full[st], 0, row, hd);
            tma_load_3d(sk + G::STAGE_BYTES / 2, m, &bars.kv_full[st], 64, row, hd);
        }
        const CUtensorMap* m = lowbit ? &maps.vh16 : (vl ? &maps.vvl : &maps.v16);
        tma_load_3d(sv, m, &bars.kv_full[st], 0, row, hd);
        tma_load_3d(sv + G::STAGE_BYTES / 2, m, &bars.kv_full[st], 64, row, hd);
    }
    if (!ok || *abort_flag) {
        // leaving early: wait (bounded) for the copies still on their way into this CTA's shared memory
        mbar_wait_sleepy(&bars.q_full, 0, limit);
        for (int u = max(t - w.t0 - NST, 0); u < t - w.t0; ++u) mbar_wait_sleepy(&bars.kv_full[u % NST], (u / NST) & 1, limit);
    } else if (settle) {
        // every stage released for the last time: no arrival is on its way to a ring barrier any more (the CTA goes on
        // to another piece of work on re-initialised barriers)
        for (int u = max(t - w.t0 - NST, 0); u < t - w.t0; ++u)
            if (!mbar_wait_sleepy(&bars.kv_free[u % NST], (u / NST) & 1, limit)) { ok = false; break; }
    }
    return ok;
}

// ---- softmax warps -------------------------------------------------------------------------------
// One thread per query row: the thread reads its 64 scores of a tile in two register halves, raises the row's
// reference when the tile's maximum exceeds it by more than the threshold (rescaling O and the row sum), and writes the
// 64 probabilities as fp16 pairs over the first 32 columns of the buffer it read.
constexpr int TC_THREADS = 384;                     // TMA producer, 2 MMA issuers, 1 idle warp, 8 softmax warps
constexpr float P_SUM_LIMIT = 65504.0f;             // a tile's row sum below the largest fp16 number: none of its P overflowed
constexpr int WARM_TILES = 8;                       // tiles at the start of a walk whose maximum is always looked at, and ...
constexpr float WARM_SPREAD = 6.0f;                 // ... how far apart (log2 units) their maxima may lie for the rest to go without
constexpr float RAISE_THRESHOLD = 14.0f;            // log2 units by which a tile must exceed the reference to raise it (P stays below 2^14, inside fp16)

// row maximum of 32 float scores held in registers
__device__ __forceinline__ float fmax3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ float row_max32(const uint32_t (&raw)[32]) {
    // three-input maximum: two columns per instruction
    float m0 = fmax3(__uint_as_float(raw[0]), __uint_as_float(raw[1]), __uint_as_float(raw[2]));
    float m1 = fmax3(__uint_as_float(raw[3]), __uint_as_float(raw[4]), __uint_as_float(raw[5]));
    float m2 = fmaxf(__uint_as_float(raw[6]), __uint_as_float(raw[7]));
#pragma unroll
    for (int e = 8; e < 32; e += 6) {
        m0 = fmax3(m0, __uint_as_float(raw[e]), __uint_as_float(raw[e + 1]));
        m1 = fmax3(m1, __uint_as_float(raw[e + 2]), __uint_as_float(raw[e + 3]));
        m2 = fmax3(m2, __uint_as_float(raw[e + 4]), __uint_as_float(raw[e + 5]));
    }
    return fmax3(m0, m1, m2);
}

// packed fp32 pairs (one instruction for two lanes of arithmetic; sm_100 fma / add on .f32x2)
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
    uint64_t v;
    asm("mov.b64 %0, {%1, %2};" : "=l"(v) : "f"(lo), "f"(hi));
    return v;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v)); }
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}

// exponentials of 32 float scores: pk receives the fp16 pairs of 2^(raw * sc + bias); returns their fp32 sum.
// Scale-and-shift and the row sum go through the packed fp32 pipe (two columns per instruction).
__device__ __forceinline__ float row_exp32(const uint32_t (&raw)[32], float sc, float bias, uint32_t (&pk)[16]) {
    const uint64_t sc2 = pack2(sc, sc), bias2 = pack2(bias, bias);
    uint64_t acc0 = pack2(0.0f, 0.0f), acc1 = acc0;
#pragma unroll
    for (int e = 0; e < 32; e += 4) {
        float x0, x1, x2, x3;
        unpack2(fma2(pack2(__uint_as_float(raw[e]), __uint_as_float(raw[e + 1])), sc2, bias2), x0, x1);
        unpack2(fma2(pack2(__uint_as_float(raw[e + 2]), __uint_as_float(raw[e + 3])), sc2, bias2), x2, x3);
        const float p0 = ex2f(x0), p1 = ex2f(x1), p2 = ex2f(x2), p3 = ex2f(x3);
        acc0 = add2(acc0, pack2(p0, p1));
        acc1 = add2(acc1, pack2(p2, p3));
        const __half2 h01 = __floats2half2_rn(p0, p1), h23 = __floats2half2_rn(p2, p3);
        pk[e >> 1] = *reinterpret_cast<const uint32_t*>(&h01);
        pk[(e >> 1) + 1] = *reinterpret_cast<const uint32_t*>(&h23);
    }
    float s0, s1, s2, s3;
    unpack2(acc0, s0, s1);
    unpack2(acc1, s2, s3);
    return (s0 + s1) + (s2 + s3);
}

// columns [c0, c0 + 32) of a boundary tile: entries outside [lo_eff, lo_eff + span] of this row become `knock`
__device__ __forceinline__ void mask_cols32(uint32_t (&raw)[32], int c0, int lo_eff, unsigned span, uint32_t knock) {
#pragma unroll
    for (int e = 0; e < 32; ++e) raw[e] = ((unsigned)(c0 + e - lo_eff) <= span) ? raw[e] : knock;
}

// LOWBIT_FP8: the low-bit codes are e4m3 bytes (kind::f8f6f4), else int8 (kind::i8).  QUERY_BLOCK: the query rows
// are the last Lq < L positions (a compile-time zero offset keeps one register out of the whole-prefill loop:
// 2.6 % on the benchmark workload).
// SPLIT (short query blocks only): several CTAs share a pair of query tiles, each on a contiguous slice of the
// walk; they leave unnormalised partial results that attn_merge_kernel combines by their reference maxima.
// EXACT = false is the kernel of the first launch: one CTA per block index.  After the first tiles of a row's low-bit pass
// (and if their maxima lie close together) it takes the exponentials against the row's reference as it stands, without
// looking for the tile's maximum, and every tile's row sum tells afterwards whether that was safe (no P beyond fp16).  If it was not for any row of the
// CTA - a score more than 2^16 above everything the row had seen - the CTA writes no output and puts its block
// index on a list.  EXACT = true is the kernel of the second launch, a small grid that goes through that list
// (normally empty) with the maximum looked at in every tile.
template <bool LOWBIT_FP8, bool QUERY_BLOCK, bool SPLIT = false, bool EXACT = false>
__global__ void __launch_bounds__(TC_THREADS, 1)
attn_tc_kernel(const __grid_constant__ TcMaps maps, const TcParams p) {
    constexpr int TBN = 64, BN = 64;
    if (EXACT && p.redo[0] == 0u) return;
    using G = Geo<TBN>;
    constexpr int NST = G::NST;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    __shared__ TcBarriers bars;
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s, restart_s, cnt_b_s[QT];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (warp == 0) {
        tmem_alloc(&tmem_base_s, TM_COLS);
        tmem_relinquish();
    }
    if (threadIdx.x == 0) abort_s = 0;
    const uint32_t n_items = EXACT ? p.redo[0] : 1u;
#pragma unroll 1
    for (uint32_t item = EXACT ? blockIdx.x : 0u; item < n_items; item += (EXACT ? gridDim.x : 1u)) {
    const int bx = EXACT ? (int)p.redo[1 + 3 * item] : (int)blockIdx.x;
    const int h = EXACT ? (int)p.redo[2 + 3 * item] : (int)blockIdx.y, b = EXACT ? (int)p.redo[3 + 3 * item] : (int)blockIdx.z;
    const int pt_lin = p.grid_x - 1 - bx;                    // pair of query tiles (and slice); longest rows first
    const int pt = SPLIT ? pt_lin / p.splits : pt_lin;
    const int split = SPLIT ? pt_lin % p.splits : 0;
    const int L = p.Lq, W = p.window, g = p.Hq / p.Hkv;     // L: rows of the query block
    const int off = QUERY_BLOCK ? p.L - p.Lq : 0;           // position of query row 0 among the keys
    const long long limit = p.wait_limit;
    // Last low-bit-eligible key position of the row at position x: x - W with the per-row sliding window,
    // min(x, L_K - W - 1) with the fixed tail window (both as min(x, lim) - wsub).  Its window keys start right
    // after it, and the vertical keys it may use are those at or below it.
    const int q_lim = (QUERY_BLOCK && p.fixed_tail) ? p.L - W - 1 : 0x7fffffff;
    const int q_sub = (QUERY_BLOCK && p.fixed_tail) ? 0 : W;
    auto qhi = [&](int x) -> int { return QUERY_BLOCK ? min(x, q_lim) - q_sub : x - W; };
    const int qhead = b * p.Hq + h, kvhead = b * p.Hkv + h / g;
    const int32_t* idx_row = p.vl_idx + (long)qhead * p.k;

    if (threadIdx.x == 0) {
        mbar_init(&bars.q_full, 1);
        for (int s = 0; s < NST; ++s) {
            mbar_init(&bars.kv_full[s], 1);
            mbar_init(&bars.kv_free[s], QT);
        }
        for (int q = 0; q < QT; ++q) {
            for (int bf = 0; bf < 2; ++bf) {
                mbar_init(&bars.s_full[q][bf], 1);
                mbar_init(&bars.p_full[q][bf], 4);                  // one arrival per softmax warp of the query tile
                mbar_init(&bars.o_done[q][bf], 1);
            }
            mbar_init(&bars.drain[q], 1);
        }
        fence_mbar_init();
        restart_s = 0;
        if (EXACT) atomicAdd(&g_tc_restarts, 1ull);
    }
    if (threadIdx.x < QT) {
        const int a1 = off + min(pt * QT * BM + (int)threadIdx.x * BM + BM - 1, L - 1);
        cnt_b_s[threadIdx.x] = (p.k > 0 && qhi(a1) >= 0) ? count_le(idx_row, p.k, qhi(a1)) : 0;
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_base_s;

    auto make_sched = [&](int q) {
        QSched s;
        s.i0 = (pt * QT + q) * BM;
        s.live = s.i0 < L;
        s.i1 = min(s.i0 + BM - 1, L - 1);
        const int a0 = s.i0 + off, a1 = s.i1 + off;             // positions of the tile's first and last row
        s.nA = (s.live && qhi(a1) >= 0) ? qhi(a1) / BN + 1 : 0;
        s.nB = s.live ? (cnt_b_s[q] + BN - 1) / BN : 0;
        s.tC0 = max(0, qhi(a0) + 1) / BN;
        s.tC1 = (s.live && W > 0) ? a1 / BN : -1;
        return s;
    };
    const QSched qs0 = make_sched(0), qs1 = make_sched(1);
    Walk w;
    w.nA = max(qs0.nA, qs1.nA);
    w.nB = max(qs0.nB, qs1.nB);
    w.tC0 = qs0.tC0;
    w.nC = (W > 0) ? max(qs0.tC1, qs1.tC1) - w.tC0 + 1 : 0;
    w.T = w.nA + w.nB + w.nC;
    w.t0 = SPLIT ? (int)((long)w.T * split / p.splits) : 0;
    w.t1 = SPLIT ? (int)((long)w.T * (split + 1) / p.splits) : w.T;

    // vertical-line keys of the low-bit pass: with e4m3 scores an extra MMA step per tile adds -inf to their columns
    const uint8_t* vl_tiles_head = (LOWBIT_FP8 && p.vl_tiles) ? p.vl_tiles + (long)qhead * (p.mask_words / 2) * VL_TILE_BYTES : nullptr;
    if (vl_tiles_head) {
        // the constant operand of that step, one copy per ring slot whose first tile is a low-bit tile (the copy of a
        // slot is overwritten by the slot's first full-precision tile, after which the slot holds no low-bit tile again)
        const int n_slots = min(min(w.nA, w.t1) - w.t0, NST);
        for (int c = threadIdx.x; c < n_slots * (int)(ONES_BYTES / 16); c += TC_THREADS) {
            const int slot = c / (int)(ONES_BYTES / 16), chunk = c % (int)(ONES_BYTES / 16);   // chunks 0..127: element 0..15 of row `chunk`
            *reinterpret_cast<uint4*>(smem + SK_OFF + slot * G::STAGE_BYTES + ONES_OFF + chunk * 16) =
                make_uint4(chunk < BM ? 0x3Cu : 0u, 0u, 0u, 0u);                               // 0x3C = 1.0 in e5m2
        }
        fence_proxy_async();
    }
    __syncthreads();

    volatile int* abort_flag = &abort_s;
    volatile int* restart_flag = &restart_s;
    auto fail = [&]() {
        *abort_flag = 1;
        if (p.status) atomicExch(p.status, HYQ_ERR_TIMEOUT);
    };

    // the single-thread roles sit in the lowest warps (the softmax warps 4..19 keep warp % 4 = TMEM lane quarter)
    if (warp == 0) {
        if (lane == 0 && !tma_producer<TBN>(maps, qs0, qs1, w, qhead, kvhead, bars, smem, abort_flag, limit, p.drop_load, vl_tiles_head, EXACT)) fail();
    } else if (warp == 1 || warp == 2) {
        if (lane == 0) {
            const int q = warp - 1;
            const bool ok = mma_issuer<LOWBIT_FP8, TBN>(q, q ? qs1 : qs0, w, bars, smem, tmem, abort_flag, limit, vl_tiles_head != nullptr);
            if (EXACT || !ok || *abort_flag) {
                // leaving early, or going on to another piece of work: none of this thread's MMAs, and none of their
                // arrivals at barriers, may be on its way when the CTA gives up its tensor memory or initialises its barriers again
                umma_commit(&bars.drain[q]);
                if (!mbar_wait(&bars.drain[q], 0, limit) && ok) fail();
            }
            if (!ok) fail();
        }
    } else if (warp >= 4) {
        // ------------------------------------------------------------------ softmax warps
        const int q = (warp - 4) >> 2;                          // query tile (a thread owns all 64 columns of its row)
        const QSched sq = q ? qs1 : qs0;
        const OwnTiles own = own_tiles(sq, w);
        // first launch: the CTA's eight softmax warps agree whether any row's exponentials overflowed; if so the CTA's
        // block index goes on the list of the second launch and nothing is written
        auto agree = [&](bool over_any) -> bool {
            if (EXACT) return false;
            if (__any_sync(0xffffffffu, over_any) && lane == 0) *restart_flag = 1;
            bar_sync_named(1, 8 * 32);
            const bool again = *restart_flag != 0 && *abort_flag == 0;
            if (again && warp == 4 && lane == 0) {
                const uint32_t slot = atomicAdd(p.redo, 1u);
                p.redo[1 + 3 * slot] = (uint32_t)bx;
                p.redo[2 + 3 * slot] = (uint32_t)h;
                p.redo[3 + 3 * slot] = (uint32_t)b;
            }
            return again;
        };
        // own tiles of this CTA: numbers [n0, n_total) in the query tile's own list (all of it unless the keys are split)
        const int n0 = SPLIT ? own_before(own, w.t0) : 0;
        const int n_total = SPLIT ? own_before(own, w.t1) : own.a_end + (own.b_end - own.b_beg) + (own.c_end - own.c_beg);
        if (SPLIT && sq.live && n_total <= n0) {
            // nothing of this query tile lies in the slice: an empty partial result
            const int i = sq.i0 + (warp & 3) * 32 + lane;
            if (i < L)
                reinterpret_cast<float2*>(p.part_ml)[((long)split * p.Hq * p.B + qhead) * L + i] = make_float2(-INFINITY, 0.0f);
        }
        if (sq.live && n_total > n0) {
            const int r = (warp & 3) * 32 + lane;               // query row inside the tile = TMEM lane
            const int i = sq.i0 + r;                           // row of the query block ...
            const int ia = i + off;                             // ... and its position among the keys
            const bool row_live = i < L;
            const bool ragged = sq.i0 + BM > L;
            const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
            const uint32_t to = tmem + tm_o(q) + lane_addr, ts0 = tmem + tm_s(q) + lane_addr;
#if HYQ_TC_VARIANT_BT
            const int bsh = p.bt_shift;
            const float q_scale = row_live ? __ldg(p.q_scales + (long)qhead * p.nbq + (i >> bsh)) : 0.0f;
#else
            const float q_scale = row_live ? __ldg(p.q_scales + (long)qhead * p.nbq + i / HYQ_BLOCK_TOKENS) : 0.0f;
#endif
            constexpr uint32_t knock_lq = LOWBIT_FP8 ? KNOCKOUT_F32 : KNOCKOUT_S32;
            float m_used = -INFINITY, l_h = 0.0f;               // reference maximum of the row; row sum
            bool over = false;                                  // a tile taken without its maximum had a row sum beyond fp16
            bool dead = false;                                  // this warp ran into an expired wait
            bool aborted = false;

            // walk position of own tile number n
            auto walk_pos = [&](int n) -> int {
                if (n < own.a_end) return n;
                const int tb = own.b_beg + (n - own.a_end);
                return (tb < own.b_end) ? tb : own.c_beg + (n - own.a_end - (own.b_end - own.b_beg));
            };
            // K scale and this half's vertical-line bitmask word of a low-bit tile, fetched one tile ahead of their use
            // (tile n of the low-bit pass sits at walk position n; its block and mask words exist for n < a_end)
#if HYQ_TC_VARIANT_BT
            // a 64-key tile n lies in block n / 2 (128-token blocks) or in blocks 2n and 2n + 1, one per column half (32)
            const float* ks_ptr = p.k_scales + (long)kvhead * p.nb;
#else
            const float* ks_ptr = p.k_scales + (long)kvhead * p.nb;
#endif
            const uint32_t* vl_ptr = p.vl_bits + (long)qhead * p.mask_words;
            float nks = 0.0f;
#if HYQ_TC_VARIANT_BT
            float nks_b = 0.0f, cs_hi = 0.0f;                   // K scale and score factor of columns 32-63 (32-token blocks: their own block)
#endif
            uint64_t nvl = 0u;                                  // both mask words of the tile (columns 0-31 low, 32-63 high)
            auto prefetch_tile = [&](int n) {
                nks = 0.0f; nvl = 0u;
#if HYQ_TC_VARIANT_BT
                nks_b = 0.0f;
#endif
                if (n >= own.a_end) return;
#if HYQ_TC_VARIANT_BT
                nks = __ldg(ks_ptr + ((n << 6) >> bsh));
                nks_b = (bsh == 5) ? __ldg(ks_ptr + 2 * n + 1) : nks;
#else
                nks = __ldg(ks_ptr + n);
#endif
                if (!LOWBIT_FP8) nvl = (uint64_t)__ldg(vl_ptr + 2 * n) | ((uint64_t)__ldg(vl_ptr + 2 * n + 1) << 32);
            };
            prefetch_tile(n0);
            const float qs2 = q_scale * p.scale_log2;

            // one tile of the online softmax for this thread's row: all 64 columns, in two register halves.  Returns
            // false when this warp ran into an expired wait.
            float tile_max = -INFINITY;                         // maximum of the tile last looked at (this row, log2 units)
            auto do_tile = [&](auto range_tag, int n, float cs, uint64_t vl, bool int_scores, int lo_eff, unsigned span) -> bool {
                constexpr bool NEED_RANGE = decltype(range_tag)::value;
                const uint32_t knock = int_scores ? KNOCKOUT_S32 : KNOCKOUT_F32;
                const int nl = n - n0;                          // tile number within this CTA's slice
                const int buf = nl & 1;
                const uint32_t ts = ts0 + buf * BN;
                if (!__all_sync(0xffffffffu, mbar_wait(&bars.s_full[q][buf], (uint32_t)(nl >> 1) & 1u, limit))) {
                    dead = true;
                    return false;
                }
                tc_fence_after();
                // vertical-line keys of a low-bit tile: -inf into their S columns before the row is read
                if (!LOWBIT_FP8 && vl != 0ull) {                 // uniform over the warp (e4m3 scores: the issuer's extra MMA step did it)
                    while (vl) { const int c = __ffsll((long long)vl) - 1; vl &= vl - 1; tmem_st1(ts + c, knock_lq); }
                    tmem_wait_st();
                }
                uint32_t ra[32], rb[32];
                tmem_ld32(ts, ra);
                tmem_ld32(ts + 32, rb);
                tmem_wait_ld();
                if (NEED_RANGE) {
                    mask_cols32(ra, 0, lo_eff, span, knock);
                    mask_cols32(rb, 32, lo_eff, span, knock);
                }
                // integer scores become the floats 2^23 + 2^22 + s by one integer add each (knocked-out entries
                // become -inf); the offset is taken out again by the bias of the exponent
                if (int_scores) {
#pragma unroll
                    for (int e = 0; e < 32; ++e) { ra[e] += INT_MAGIC; rb[e] += INT_MAGIC; }
                }
#if HYQ_TC_VARIANT_BT
                const float csb = cs_hi;                        // the second half's factor (its own K scale with 32-token blocks)
#endif
                {
#if HYQ_TC_VARIANT_BT
                const float fa = row_max32(ra) - (int_scores ? INT_MAGIC_F : 0.0f), fb = row_max32(rb) - (int_scores ? INT_MAGIC_F : 0.0f);
                const float mt = fmaxf((fa == -INFINITY) ? -INFINITY : fa * cs, (fb == -INFINITY) ? -INFINITY : fb * csb);
#else
                const float f = fmaxf(row_max32(ra), row_max32(rb)) - (int_scores ? INT_MAGIC_F : 0.0f);
                const float mt = (f == -INFINITY) ? -INFINITY : f * cs;
#endif
                tile_max = mt;
                const bool raise = mt > m_used + RAISE_THRESHOLD;
                if (__any_sync(0xffffffffu, raise)) {
                    const float alpha = raise ? ex2f(m_used - mt) : 1.0f;      // m_used = -inf -> 0
                    if (nl > 0) {
                        // P.V of tile n-1 must have landed before O is rescaled.  P.V number m signals barrier m & 1;
                        // the one before the previous is complete (the scores just read were issued after it), so
                        // the parity wait cannot alias.
                        if (!__all_sync(0xffffffffu, mbar_wait(&bars.o_done[q][(nl - 1) & 1], (uint32_t)((nl - 1) >> 1) & 1u, limit))) {
                            dead = true;
                            return false;
                        }
                        tc_fence_after();
#pragma unroll 1
                        for (int c = 0; c < 8; ++c) {
                            uint32_t o[16];
                            tmem_ld16(to + c * 16, o);
                            tmem_wait_ld();
#pragma unroll
                            for (int e = 0; e < 16; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
                            tmem_st16(to + c * 16, o);
                        }
                        tmem_wait_st();
                    }
                    if (raise) {
                        l_h *= alpha;
                        m_used = mt;
                    }
                }
                }
                // ---- P = 2^(s - m) as fp16 pairs over the first 32 columns of the buffer; row sum
                const float m_eff = (m_used == -INFINITY) ? 0.0f : m_used;
                const float bias = int_scores ? fmaf(-INT_MAGIC_F, cs, -m_eff) : -m_eff;
                uint32_t pa[16], pb[16];
                const float t_a = row_exp32(ra, cs, bias, pa);
                tmem_st16(ts, pa);
#if HYQ_TC_VARIANT_BT
                const float t_b = row_exp32(rb, csb, int_scores ? fmaf(-INT_MAGIC_F, csb, -m_eff) : -m_eff, pb);
#else
                const float t_b = row_exp32(rb, cs, bias, pb);
#endif
                l_h += t_a + t_b;
                tmem_st16(ts + 16, pb);
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&bars.p_full[q][buf]);
                return true;
            };

            // ---- low-bit tiles that lie wholly below every row's window: no range mask, no bounds to compute
            const int n_plain = ragged ? 0 : min(own.a_end, max(0, (qhi(sq.i0 + off) + 1) / BN));
            int n = n0;
            // First launch: the first WARM_TILES tiles are looked at in full.  If the maxima of these tiles lie close together
            // for every row of the warp (scores without heavy tails: none of the later ones will be 2^16 above the reference),
            // the plain tiles that follow go without their maximum; a warp with a row whose tile maxima spread out keeps
            // looking (such rows raise their reference often, and a second pass over the whole CTA would cost more).
            bool warm = false;
            const int n_plain_end = min(n_plain, n_total);
            auto plain_tile = [&]() -> bool {
                // a zero scale (all-zero tile) still has to let -inf pass through the multiply
                const float cs = fmaxf(qs2 * nks, 1e-37f);
#if HYQ_TC_VARIANT_BT
                cs_hi = fmaxf(qs2 * nks_b, 1e-37f);
#endif
                const auto vl = nvl;
                prefetch_tile(n + 1);
                return do_tile(std::false_type{}, n, cs, vl, !LOWBIT_FP8, 0, 0u);
            };
            if (!EXACT && n_plain_end - n0 > WARM_TILES) {
                float mt_lo = INFINITY, mt_hi = -INFINITY;
                for (; n < n0 + WARM_TILES; ++n) {
                    if (!plain_tile()) { aborted = true; break; }
                    mt_lo = fminf(mt_lo, tile_max);
                    mt_hi = fmaxf(mt_hi, tile_max);
                }
                warm = !aborted && __all_sync(0xffffffffu, m_used > -INFINITY && mt_hi - mt_lo < WARM_SPREAD);
            }
            if (!warm) {
                for (; n < n_plain_end && !aborted; ++n)
                    if (!plain_tile()) { aborted = true; break; }
            }
            if (!EXACT && warm && !aborted) {
                // Steady state of the first launch: exponentials against the reference as it stands.  The first half of a
                // tile's scores is read while the previous tile's second half is still being worked on (when the scores
                // are there by then), the second half under the first half's exponentials.
                const int n_end = n_plain_end;
                uint32_t ra[32], rb[32];
                bool have_a = false;
                for (; n < n_end; ++n) {
                    const float cs = fmaxf(qs2 * nks, 1e-37f);
#if HYQ_TC_VARIANT_BT
                    const float csb = fmaxf(qs2 * nks_b, 1e-37f);
#else
                    const float csb = cs;
#endif
                    uint64_t vl = nvl;                         // this tile's vertical-line columns (integer scores only)
                    prefetch_tile(n + 1);
                    const int nl = n - n0, buf = nl & 1;
                    const uint32_t ts = ts0 + buf * BN;
                    if (!have_a) {
                        if (!__all_sync(0xffffffffu, mbar_wait(&bars.s_full[q][buf], (uint32_t)(nl >> 1) & 1u, limit))) { dead = true; aborted = true; break; }
                        tc_fence_after();
                        if (!LOWBIT_FP8 && vl != 0ull) {
                            while (vl) { const int c = __ffsll((long long)vl) - 1; vl &= vl - 1; tmem_st1(ts + c, knock_lq); }
                            tmem_wait_st();
                        }
                        tmem_ld32(ts, ra);
                    }
                    tmem_wait_ld();
                    tmem_ld32(ts + 32, rb);
                    if (!LOWBIT_FP8) {
#pragma unroll
                        for (int e = 0; e < 32; ++e) ra[e] += INT_MAGIC;
                    }
                    const float bias = LOWBIT_FP8 ? -m_used : fmaf(-INT_MAGIC_F, cs, -m_used);
                    const float bias_b = LOWBIT_FP8 ? -m_used : fmaf(-INT_MAGIC_F, csb, -m_used);
                    uint32_t pa[16], pb[16];
                    const float t_a = row_exp32(ra, cs, bias, pa);
                    tmem_st16(ts, pa);
                    tmem_wait_ld();
                    have_a = false;
                    if (n + 1 < n_end) {
                        const int nl1 = nl + 1, buf1 = nl1 & 1;
                        if (__all_sync(0xffffffffu, mbar_test_wait(&bars.s_full[q][buf1], (uint32_t)(nl1 >> 1) & 1u))) {
                            tc_fence_after();
                            if (!LOWBIT_FP8 && nvl != 0ull) {     // (nvl: the next tile's columns by now)
                                uint64_t v1 = nvl;
                                while (v1) { const int c = __ffsll((long long)v1) - 1; v1 &= v1 - 1; tmem_st1(ts0 + buf1 * BN + c, knock_lq); }
                                tmem_wait_st();
                            }
                            tmem_ld32(ts0 + buf1 * BN, ra);
                            have_a = true;
                        }
                    }
                    if (!LOWBIT_FP8) {
#pragma unroll
                        for (int e = 0; e < 32; ++e) rb[e] += INT_MAGIC;
                    }
                    const float t_b = row_exp32(rb, csb, bias_b, pb);
                    tmem_st16(ts + 16, pb);
                    l_h += t_a + t_b;
                    over |= !(t_a + t_b < P_SUM_LIMIT);
                    tmem_wait_st();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&bars.p_full[q][buf]);
                }
                if (have_a) tmem_wait_ld();
            }
            // ---- the remaining low-bit tiles, the vertical-line tiles and the window tiles
            // (number of vertical-line keys this row may use: only needed from here on)
            const int cnt_r = (!aborted && sq.nB > 0 && row_live && qhi(ia) >= 0) ? count_le(idx_row, p.k, qhi(ia)) : 0;
            for (; n < n_total && !aborted; ++n) {
                const int t = walk_pos(n);
                const float ks = nks;
#if HYQ_TC_VARIANT_BT
                const float ks_b = nks_b;
#endif
                const auto vl = nvl;
                prefetch_tile(n + 1);
                int lo = 0, hi = -1;
                float cs;
                const bool lowbit = t < own.a_end;
                if (lowbit) {
                    hi = row_live ? min(qhi(ia) - t * BN, BN - 1) : -1;
                    cs = fmaxf(qs2 * ks, 1e-37f);
                } else if (t < own.b_end) {
                    hi = min(cnt_r - (t - own.b_beg) * BN - 1, BN - 1);
                    cs = p.scale_log2;
                } else {
                    const int j0 = (w.tC0 + t - w.nA - w.nB) * BN;
                    lo = max(0, qhi(ia) + 1 - j0);
                    hi = row_live ? min(ia - j0, BN - 1) : -1;
                    cs = p.scale_log2;
                }
#if HYQ_TC_VARIANT_BT
                cs_hi = lowbit ? fmaxf(qs2 * ks_b, 1e-37f) : cs;
#endif
                const int lo_eff = (hi >= lo) ? lo : 4096;
                const unsigned span = (hi >= lo) ? (unsigned)(hi - lo) : 0u;
                // tiles that every row of this warp uses in full (most window and vertical-line tiles) need no range mask
                // (with two threads per row both warps of a pair still meet at the same named barriers)
                if (__all_sync(0xffffffffu, lo == 0 && hi == BN - 1)) {
                    if (!do_tile(std::false_type{}, n, cs, vl, lowbit && !LOWBIT_FP8, 0, 0u)) aborted = true;
                    continue;
                }
                if (!do_tile(std::true_type{}, n, cs, vl, lowbit && !LOWBIT_FP8, lo_eff, span)) aborted = true;
            }

            // ---- epilogue: the last P.V (MMAs complete in order), sum of the two halves' row sums, O / l
            bool ok = !aborted && !dead;
            if (ok) ok = __all_sync(0xffffffffu, mbar_wait(&bars.o_done[q][(n_total - n0 - 1) & 1], (uint32_t)((n_total - n0 - 1) >> 1) & 1u, limit));
            const bool again = agree(over);
            if (!aborted && !again) {                           // uniform over the query tile's softmax warps
                tc_fence_after();
                constexpr int NCH = 4;                          // 32-channel pieces of the row this thread writes
                const float l_run = l_h;
                const float inv = (l_run > 0.0f) ? 1.0f / l_run : 0.0f;
                if (SPLIT) {
                    // partial result of this slice: O as accumulated (relative to m_used), the pair (m_used, l)
                    const long prow = ((long)split * p.Hq * p.B + qhead) * L + i;
                    if (ok) {
#pragma unroll
                        for (int c = 0; c < NCH; ++c) {
                            uint32_t o[32];
                            const int ch = c * 32;
                            tmem_ld32(to + ch, o);
                            tmem_wait_ld();
                            if (row_live) {
                                uint4* dst = reinterpret_cast<uint4*>(p.part_o + prow * HYQ_D + ch);
#pragma unroll
                                for (int e = 0; e < 8; ++e) dst[e] = make_uint4(o[4 * e], o[4 * e + 1], o[4 * e + 2], o[4 * e + 3]);
                            }
                        }
                        if (row_live) reinterpret_cast<float2*>(p.part_ml)[prow] = make_float2(m_used, l_run);
                    }
                } else if (ok) {
#pragma unroll
                    for (int c = 0; c < NCH; ++c) {
                        uint32_t o[32];
                        const int ch = c * 32;
                        tmem_ld32(to + ch, o);
                        tmem_wait_ld();
                        if (row_live) {
                            if (p.out_fp32) {
                                float4* dst = reinterpret_cast<float4*>(static_cast<float*>(p.out) + ((long)qhead * L + i) * HYQ_D + ch);
#pragma unroll
                                for (int e = 0; e < 8; ++e)
                                    dst[e] = make_float4(__uint_as_float(o[4 * e]) * inv, __uint_as_float(o[4 * e + 1]) * inv,
                                                         __uint_as_float(o[4 * e + 2]) * inv, __uint_as_float(o[4 * e + 3]) * inv);
                            } else {
                                uint4* dst = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(p.out) + ((long)qhead * L + i) * HYQ_D + ch);
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    uint32_t wd[4];
#pragma unroll
                                    for (int q2 = 0; q2 < 4; ++q2) {
                                        const __nv_bfloat162 b2 = __floats2bfloat162_rn(__uint_as_float(o[8 * e + 2 * q2]) * inv,
                                                                                        __uint_as_float(o[8 * e + 2 * q2 + 1]) * inv);
                                        wd[q2] = *reinterpret_cast<const uint32_t*>(&b2);
                                    }
                                    dst[e] = make_uint4(wd[0], wd[1], wd[2], wd[3]);
                                }
                            }
                        }
                    }
                    if (p.lse && row_live) p.lse[(long)qhead * L + i] = (m_used + log2f(l_run)) * 0.6931471805599453f;
                }
            }
            if (!ok) fail();
        } else {
            agree(false);                                       // (a query tile with nothing to do still takes part)
        }
    }

    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (EXACT && abort_s) break;
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        __syncwarp();
        tmem_dealloc(tmem_base_s, TM_COLS);
    }
}

// Combines the partial results of the key slices of a short query block: every slice s left, per row, its
// accumulator O_s relative to its own reference maximum m_s (log2 units) and its row sum l_s; the row's result is
// sum_s 2^(m_s - M) O_s / sum_s 2^(m_s - M) l_s with M = max_s m_s.  One thread per row and four channels.
__global__ void __launch_bounds__(256)
attn_merge_kernel(const float* __restrict__ part_o, const float* __restrict__ part_ml, int splits, long n_rows, void* out,
                  int out_fp32, float* lse) {
    const long e = (long)blockIdx.x * blockDim.x + threadIdx.x;
    const long row = e / (HYQ_D / 4);
    const int c4 = (int)(e % (HYQ_D / 4));
    if (row >= n_rows) return;
    float m = -INFINITY;
    for (int s = 0; s < splits; ++s) m = fmaxf(m, __ldg(part_ml + ((long)s * n_rows + row) * 2));
    float4 acc = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
    float l = 0.0f;
    for (int s = 0; s < splits; ++s) {
        const float2 ml = __ldg(reinterpret_cast<const float2*>(part_ml) + (long)s * n_rows + row);
        if (!(ml.y > 0.0f)) continue;                           // empty slice: its accumulator was not written
        const float wgt = exp2f(ml.x - m);
        const float4 o = __ldg(reinterpret_cast<const float4*>(part_o + ((long)s * n_rows + row) * HYQ_D) + c4);
        acc.x = fmaf(wgt, o.x, acc.x); acc.y = fmaf(wgt, o.y, acc.y); acc.z = fmaf(wgt, o.z, acc.z); acc.w = fmaf(wgt, o.w, acc.w);
        l = fmaf(wgt, ml.y, l);
    }
    const float inv = (l > 0.0f) ? 1.0f / l : 0.0f;
    acc.x *= inv; acc.y *= inv; acc.z *= inv; acc.w *= inv;
    if (out_fp32) {
        reinterpret_cast<float4*>(static_cast<float*>(out) + row * HYQ_D)[c4] = acc;
    } else {
        const __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y), hi = __floats2bfloat162_rn(acc.z, acc.w);
        reinterpret_cast<uint2*>(static_cast<__nv_bfloat16*>(out) + row * HYQ_D)[c4] =
            make_uint2(*reinterpret_cast<const uint32_t*>(&lo), *reinterpret_cast<const uint32_t*>(&hi));
    }
    if (lse && c4 == 0) lse[row] = (m + log2f(l)) * 0.6931471805599453f;
}

// ---------------------------------------------------------------------------------------------
size_t attn_tc_workspace_bytes(const hyq_attn_args& a) { return tc_workspace_layout(a).total; }

// CTAs of this translation unit's kernels whose work was done a second time (synchronises the device)
int tc_restarts(unsigned long long* count, bool reset) {
    if (cudaMemcpyFromSymbol(count, g_tc_restarts, sizeof(*count)) != cudaSuccess) return HYQ_ERR_CUDA;
    const unsigned long long zero = 0ull;
    if (reset && cudaMemcpyToSymbol(g_tc_restarts, &zero, sizeof(zero)) != cudaSuccess) return HYQ_ERR_CUDA;
    return HYQ_OK;
}

int launch_attn_tc(const hyq_attn_args& a, float alpha, cudaStream_t st) {
    constexpr int TBN = 64;                                             // keys per tile
    const TcWorkspace w = tc_workspace_layout(a);
    const int rc = launch_tc_prepass(a, w, st);
    if (rc != HYQ_OK) return rc;
    char* base = static_cast<char*>(a.workspace);
    const bool int4 = a.q_format == HYQ_FMT_INT4;
    const uint64_t qh = (uint64_t)a.B * a.Hq, kvh = (uint64_t)a.B * a.Hkv, L = a.L, Lq = query_rows(a);
    const uint64_t kk = a.k > 0 ? a.k : 1;

    TcMaps maps;
    bool ok = true;
    ok &= make_tmap_3d(&maps.q, a.q, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, HYQ_D, Lq, qh, 64, BM);
    ok &= make_tmap_3d(&maps.k, a.k_, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, HYQ_D, L, kvh, 64, TBN);
    ok &= make_tmap_3d(&maps.qc, int4 ? (const void*)(base + w.q8) : a.q_codes, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, HYQ_D, Lq, qh, 128, BM);
    ok &= make_tmap_3d(&maps.kc, int4 ? (const void*)(base + w.k8) : a.k_codes, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, HYQ_D, L, kvh, 128, TBN);
    ok &= make_tmap_3d(&maps.v16, base + w.v16, CU_TENSOR_MAP_DATA_TYPE_UINT16, 2, HYQ_D, L, kvh, 64, TBN);
    ok &= make_tmap_3d(&maps.vh16, base + w.vh16, CU_TENSOR_MAP_DATA_TYPE_UINT16, 2, HYQ_D, L, kvh, 64, TBN);
    ok &= make_tmap_3d(&maps.kvl, base + w.kvl, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, HYQ_D, kk, qh, 64, TBN);
    ok &= make_tmap_3d(&maps.vvl, base + w.vvl, CU_TENSOR_MAP_DATA_TYPE_UINT16, 2, HYQ_D, kk, qh, 64, TBN);
    if (!ok) return HYQ_ERR_CUDA;

    TcParams p{};
    p.B = a.B; p.Hq = a.Hq; p.Hkv = a.Hkv; p.L = a.L; p.window = a.window; p.k = a.k;
#if HYQ_TC_VARIANT_BT
    p.nb = (a.L + a.block_tokens - 1) / a.block_tokens;
    p.bt_shift = a.block_tokens == 32 ? 5 : 7;
#else
    p.nb = (a.L + HYQ_BLOCK_TOKENS - 1) / HYQ_BLOCK_TOKENS;
#endif
    p.Lq = (int)Lq;
    p.fixed_tail = a.window_mode == HYQ_WINDOW_FIXED_TAIL;
    p.splits = w.splits;
    p.part_o = reinterpret_cast<float*>(base + w.part_o);
    p.part_ml = reinterpret_cast<float*>(base + w.part_ml);
#if HYQ_TC_VARIANT_BT
    p.nbq = ((int)Lq + a.block_tokens - 1) / a.block_tokens;
#else
    p.nbq = ((int)Lq + HYQ_BLOCK_TOKENS - 1) / HYQ_BLOCK_TOKENS;
#endif
    p.mask_words = w.mask_words;
    p.out_fp32 = a.out_dtype == 1;
    p.scale_log2 = alpha * 1.4426950408889634f;
    p.q_scales = a.q_scales; p.k_scales = a.k_scales; p.vl_idx = a.vl_idx;
    p.vl_bits = reinterpret_cast<const uint32_t*>(base + w.vl_bits);
    p.vl_tiles = (a.q_format != HYQ_FMT_INT8 && a.k > 0) ? reinterpret_cast<const uint8_t*>(base + w.vl_tiles) : nullptr;
    p.out = a.out; p.lse = a.lse; p.status = a.status_word;
    const TcTestHooks hooks = tc_test_hooks();
    p.wait_limit = hooks.wait_limit > 0 ? hooks.wait_limit : WAIT_LIMIT_DEFAULT;
    p.drop_load = hooks.drop_load;

    const bool blk = Lq < L || p.fixed_tail;      // the general instantiation (the other one is the whole prefill)
    // e4m3 bytes on the low-bit side: FP8 codes as they are, or INT4 codes widened by the pre-pass
    const bool lowbit_fp8 = a.q_format != HYQ_FMT_INT8;
    const bool split = w.splits > 1;               // (only ever chosen for short query blocks)
    auto kern = split ? (lowbit_fp8 ? attn_tc_kernel<true, true, true> : attn_tc_kernel<false, true, true>)
              : lowbit_fp8 ? (blk ? attn_tc_kernel<true, true> : attn_tc_kernel<true, false>)
                           : (blk ? attn_tc_kernel<false, true> : attn_tc_kernel<false, false>);
    // the same instantiation for the second launch (every maximum looked at; works through the first launch's list)
    auto kern_exact = split ? (lowbit_fp8 ? attn_tc_kernel<true, true, true, true> : attn_tc_kernel<false, true, true, true>)
                    : lowbit_fp8 ? (blk ? attn_tc_kernel<true, true, false, true> : attn_tc_kernel<true, false, false, true>)
                                 : (blk ? attn_tc_kernel<false, true, false, true> : attn_tc_kernel<false, false, false, true>);
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)TC_SMEM_BYTES) != cudaSuccess ||
        cudaFuncSetAttribute(kern_exact, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)TC_SMEM_BYTES) != cudaSuccess)
        return HYQ_ERR_CUDA;
    const dim3 grid((((int)Lq + QT * BM - 1) / (QT * BM)) * w.splits, a.Hq, a.B);
    p.grid_x = (int)grid.x;
    p.redo = reinterpret_cast<uint32_t*>(base + w.redo);
    if (cudaMemsetAsync(p.redo, 0, sizeof(uint32_t), st) != cudaSuccess) return HYQ_ERR_CUDA;
    if (a.ev_kernel_start && cudaEventRecord(static_cast<cudaEvent_t>(a.ev_kernel_start), st) != cudaSuccess) return HYQ_ERR_CUDA;
    kern<<<grid, TC_THREADS, TC_SMEM_BYTES, st>>>(maps, p);
    if (launch_status() != HYQ_OK) return HYQ_ERR_CUDA;
    const long n_ctas = (long)grid.x * grid.y * grid.z;
    {
        kern_exact<<<(unsigned)(n_ctas < 148 ? n_ctas : 148), TC_THREADS, TC_SMEM_BYTES, st>>>(maps, p);
        if (launch_status() != HYQ_OK) return HYQ_ERR_CUDA;
    }
    if (split) {
        const long n_rows = (long)a.B * a.Hq * (long)Lq, n_thr = n_rows * (HYQ_D / 4);
        attn_merge_kernel<<<(unsigned)((n_thr + 255) / 256), 256, 0, st>>>(p.part_o, p.part_ml, w.splits, n_rows, a.out, p.out_fp32, a.lse);
        if (launch_status() != HYQ_OK) return HYQ_ERR_CUDA;
    }
    if (a.ev_kernel_stop && cudaEventRecord(static_cast<cudaEvent_t>(a.ev_kernel_stop), st) != cudaSuccess) return HYQ_ERR_CUDA;
    return HYQ_OK;
}

#if HYQ_TC_VARIANT_BT
}  // namespace tcbt
#endif
}  // namespace hyq
