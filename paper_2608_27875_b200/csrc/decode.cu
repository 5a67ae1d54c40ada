// Hybrid-precision KV-cache attention for one new token (Algorithm 3 / Section 3.3).
//
// The op is a stream over the cache: every cached row is read once, 128 B per INT4 row (K + V) and 512 B per
// bf16 row, against 2 * g * 128 multiply-adds per row and tensor - HBM-bound once the arithmetic is cheap
// enough.  With g = 4 query heads per KV head, CUDA-core FMAs plus the nibble unpacking would need more
// issue slots than the memory system leaves time for, and a tcgen05 path would have to write the
// dequantized tile to shared memory first (4x the bytes that came from HBM, more than the shared-memory
// bandwidth that 1/148th of 7 TB/s allows).  So the codes are dequantized in registers, straight into the
// operand layout of the warp-level matrix instruction (mma.sync m16n8k16, fp32 accumulate), with the long
// side of the instruction on the keys (Q.K^T) or the channels (P.V) and the 8-wide side on the g heads:
//
//   S^T[16 keys x 8 heads]   = Khat[16 x 128] . q^T            8 k-steps; A from the codes, B from q (fp16)
//   O^T[128 ch  x 8 heads]  += Vhat^T[128 x 16] . P^T[16 x 8]  8 m-tiles; A from the codes, B = P^T
//
// The contraction index of the first product and the row index of the second may be permuted freely, so
// each lane takes whatever channels arrive in its own 16-byte loads; P^T's operand layout is the transpose
// of S^T's accumulator layout, which `movmatrix` provides for 8x8 b16 blocks.  V's codes are stored by
// Freeze in exactly the operand order (see hyq_decode.h), K's stay row-major.  INT4 -> fp16 is one LOP3
// (nibble ^ 8 | 0x6400 = 1032 + code) and one packed subtract or fma for two codes.
// The bf16 segments (vertical rows, staging, window) go through the same two products with bf16 operands;
// there V^T's key pairs are formed from two rows' words with byte permutes.
//
// Grid: (splits, B * Hkv).  A CTA owns a contiguous slice of the head's INT4 tiles and one of its bf16 tiles
// (the three bf16 segments form one tile list); its 4 warps take tiles round-robin, each with its own online-softmax state, which
// are merged through shared memory; the slices' (m, l, acc) go to the workspace and decode_merge_kernel
// applies ReduceSoftmax.  Softmax is lazy: a tile only raises the running reference maximum when one of its
// scores exceeds it by more than 2^DEC_RAISE (warp vote), so the usual tile costs four compares, four ex2
// and no shuffle.
#include <cuda_fp16.h>

#include "decode_common.cuh"

namespace hyq {

constexpr int DEC_THREADS = 128;
constexpr int DEC_WARPS = DEC_THREADS / 32;
#ifndef DEC_CTAS_PER_SM
#define DEC_CTAS_PER_SM 4                   // resident CTAs per SM the register budget is set for
#endif
#ifndef DEC_PAIR
#define DEC_PAIR 1                           // INT4 tiles are processed two at a time
#endif
#ifndef DEC_STAGES_N
#define DEC_STAGES_N 4
#endif
constexpr int DEC_STAGES = DEC_STAGES_N;    // tiles in flight per warp (cp.async ring)
constexpr int DEC_STAGE_BYTES = 2048;       // 1 KB K codes + 1 KB V codes
constexpr float DEC_RAISE = 8.0f;          // log2 units; P <= 2^8 stays far inside fp16 / bf16 range

struct DecParams {
    int g, splits, Hkv;
    int hgroups;         // ceil(g / 8): a KV head with more than 8 query heads is served by several CTAs per slice
    int gshift;          // log2(rows per scale group / 16): 16-row tile t belongs to group t >> gshift
    long nQ, sQ;         // quantized rows per head (valid), rows between heads
    int k, W, n_s;       // valid rows of the vertical, window and staging buffers ...
    int sK, sW, Ws;      // ... and rows between heads
    const int4* lens;    // optional per-sequence {quantized, vertical, window, staging} valid rows (ragged batch)
    float scale_log2;
    const uint8_t* kq; const uint8_t* vq; const float* ks; const float* vs;
    const uint4 *k_vl, *v_vl, *k_s, *v_s, *k_win, *v_win;
    const uint4* q;
    float* part_acc;     // [unit][split][8 heads][128 channels]  unnormalised
    float* part_ml;      // [unit][split][8 heads][2]             reference maximum (log2 units), row sum
};

__device__ __forceinline__ void mma_f16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                        uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// 8x8 b16 transpose across the warp: lane 4r+j gives (row r, cols 2j, 2j+1), receives the same of the transpose
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
    uint32_t d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
    return d;
}
// Two INT4 codes (two's complement nibbles) -> packed fp16 values, without unpacking shifts where possible:
// dq4_lo takes the nibbles at bits 0-3 / 16-19: (w & 0x000F000F) ^ 0x64086408 is fp16 1032 + code, minus 1032;
// dq4_hi takes the nibbles at bits 4-7 / 20-23: (w & 0x00F000F0) ^ 0x64806480 is fp16 16 * (72 + code), so one
// packed fma (x / 16 - 72) finishes it.  Both are exact.
__device__ __forceinline__ uint32_t dq4_lo(uint32_t w) {
    uint32_t h;
    asm("lop3.b32 %0, %1, 0x000F000F, 0x64086408, 0x6A;" : "=r"(h) : "r"(w));
    asm("sub.rn.f16x2 %0, %1, %2;" : "=r"(h) : "r"(h), "r"(0x64086408u));
    return h;
}
__device__ __forceinline__ uint32_t dq4_hi(uint32_t w) {
    uint32_t h;
    asm("lop3.b32 %0, %1, 0x00F000F0, 0x64806480, 0x6A;" : "=r"(h) : "r"(w));
    asm("fma.rn.f16x2 %0, %1, %2, %3;" : "=r"(h) : "r"(h), "r"(0x2C002C00u), "r"(0xD480D480u));
    return h;
}
// K side only: the codes enter the matrix instruction as fp16 SUBNORMALS with no arithmetic at all - the nibble
// (xor 8, i.e. code + 8) placed in mantissa bits 0-3 is (code + 8) * 2^-24, placed in bits 4-7 it is
// (code + 8) * 2^-20.  The factor 16 of the second form is taken out of q's operand for those channels, the
// common 2^-24 goes into the score scale, and the +8 becomes 8 * sum_d q_d per head, subtracted from the score
// (a cancellation of a few units against a dot product of eight k-steps: harmless in fp32).  The products
// fp16 x fp16 are exact in the instruction's fp32 accumulation.
#ifndef DEC_K_SUBNORMAL
#define DEC_K_SUBNORMAL 1
#endif
__device__ __forceinline__ uint32_t kq4_lo(uint32_t w) {
#if DEC_K_SUBNORMAL
    uint32_t h;
    asm("lop3.b32 %0, %1, 0x000F000F, 0x00080008, 0x6A;" : "=r"(h) : "r"(w));
    return h;
#else
    return dq4_lo(w);
#endif
}
__device__ __forceinline__ uint32_t kq4_hi(uint32_t w) {
#if DEC_K_SUBNORMAL
    uint32_t h;
    asm("lop3.b32 %0, %1, 0x00F000F0, 0x00800080, 0x6A;" : "=r"(h) : "r"(w));
    return h;
#else
    return dq4_hi(w);
#endif
}
constexpr float DEC_K_UNIT = DEC_K_SUBNORMAL ? 16777216.0f : 1.0f;      // 2^24: undoes the subnormal placement
__device__ __forceinline__ uint32_t pack_f16(float lo, float hi) {
    uint32_t d;
    asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    uint32_t d;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}
__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// Ampere-style asynchronous 16-byte copy global -> shared (no register staging, completion by groups)
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint32_t word_of(const uint4& v, int i) {
    return i == 0 ? v.x : i == 1 ? v.y : i == 2 ? v.z : v.w;
}
// channel of accumulator row (m-tile x, lane row r, e = 0: row r, 1: row r + 8); also V's code layout
__device__ __forceinline__ int acc_channel(int x, int r, int e) { return 64 * (x >> 2) + 8 * r + 2 * (x & 3) + e; }

struct SoftmaxState {
    float m0, m1, l0, l1;      // heads 2j and 2j+1 of this lane: reference maximum (log2 units), partial row sum
};

// One tile's raw scores c4 (keys r and r+8, heads 2j and 2j+1) times f (log2 units) -> weights p[4].
// MASKED: rows flagged invalid (past the end of a segment) get weight zero.  The reference maxima are raised,
// and the accumulators rescaled, only when some score is more than 2^DEC_RAISE above them (warp vote).
// b0, b1: per-head constants subtracted from the raw scores before scaling (zero unless the K operand carries
// an offset).
template <bool MASKED>
__device__ __forceinline__ void softmax_tile(SoftmaxState& st, float (&acc)[8][4], const float (&c4)[4], float f,
                                             float b0, float b1, bool valid_a, bool valid_b, float (&p)[4]) {
    const float mm0 = fmaf(b0, f, st.m0), mm1 = fmaf(b1, f, st.m1);
    float d0 = fmaf(c4[0], f, -mm0), d2 = fmaf(c4[2], f, -mm0);
    float d1 = fmaf(c4[1], f, -mm1), d3 = fmaf(c4[3], f, -mm1);
    if (MASKED) {
        if (!valid_a) d0 = d1 = -INFINITY;
        if (!valid_b) d2 = d3 = -INFINITY;
    }
    const bool far = fmaxf(d0, d2) > DEC_RAISE || fmaxf(d1, d3) > DEC_RAISE;
    if (__any_sync(0xffffffffu, far)) {
        float s0 = (c4[0] - b0) * f, s1 = (c4[1] - b1) * f, s2 = (c4[2] - b0) * f, s3 = (c4[3] - b1) * f;
        if (MASKED) {
            if (!valid_a) s0 = s1 = -INFINITY;
            if (!valid_b) s2 = s3 = -INFINITY;
        }
        float t0 = fmaxf(s0, s2), t1 = fmaxf(s1, s3);
#pragma unroll
        for (int o = 4; o < 32; o <<= 1) {
            t0 = fmaxf(t0, __shfl_xor_sync(0xffffffffu, t0, o));
            t1 = fmaxf(t1, __shfl_xor_sync(0xffffffffu, t1, o));
        }
        const float n0 = fmaxf(st.m0, t0), n1 = fmaxf(st.m1, t1);      // finite: every tile has a valid row
        const float c0 = ex2(st.m0 - n0), c1 = ex2(st.m1 - n1);        // 0 on the first tile (m = -inf)
        st.m0 = n0; st.m1 = n1;
        st.l0 *= c0; st.l1 *= c1;
#pragma unroll
        for (int x = 0; x < 8; ++x) { acc[x][0] *= c0; acc[x][2] *= c0; acc[x][1] *= c1; acc[x][3] *= c1; }
        d0 = s0 - n0; d2 = s2 - n0; d1 = s1 - n1; d3 = s3 - n1;
    }
    p[0] = ex2(d0); p[1] = ex2(d1); p[2] = ex2(d2); p[3] = ex2(d3);
    st.l0 += p[0] + p[2];
    st.l1 += p[1] + p[3];
}

// One 16-row tile of the quantized prefix as it sits in registers: K rows r and r+8 (this lane's 16 bytes each),
// the lane's 2 x 16 bytes of the V tile, and the group's two scales.
struct QTile {
    uint4 ka, kb, va, vb;
    float fk, fv;
};

template <bool RAGGED>
__device__ __forceinline__ void quant_tile(const QTile& d, const uint32_t (&qf)[16], float scale_log2, float bias0, float bias1,
                                           int rows_valid, int r, SoftmaxState& st, float (&acc)[8][4]) {
    float c4[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
    for (int c = 0; c < 8; ++c) {
        const uint32_t wa = word_of(d.ka, c >> 1) >> (8 * (c & 1)), wb = word_of(d.kb, c >> 1) >> (8 * (c & 1));
        mma_f16(c4, kq4_lo(wa), kq4_lo(wb), kq4_hi(wa), kq4_hi(wb), qf[2 * c], qf[2 * c + 1]);
    }
    float pw[4];
    softmax_tile<RAGGED>(st, acc, c4, d.fk * scale_log2, bias0, bias1, r < rows_valid, r + 8 < rows_valid, pw);
    const uint32_t b0 = movmatrix_trans(pack_f16(pw[0] * d.fv, pw[1] * d.fv));
    const uint32_t b1 = movmatrix_trans(pack_f16(pw[2] * d.fv, pw[3] * d.fv));
#pragma unroll
    for (int x = 0; x < 8; ++x) {
        const uint32_t w = word_of(x < 4 ? d.va : d.vb, x & 3);
        mma_f16(acc[x], dq4_lo(w), dq4_hi(w), dq4_lo(w >> 8), dq4_hi(w >> 8), b0, b1);
    }
}

// Two full tiles at once: both Q.K^T chains are issued back to back and the second tile's softmax runs while the
// first tile's P.V instructions are in flight - more independent work per warp, which is what a kernel with
// few warps per SM lacks.  P.V of the first tile precedes the second softmax because that softmax may rescale
// the accumulators.
__device__ __forceinline__ void quant_tile_pair(const QTile& d0, const QTile& d1, const uint32_t (&qf)[16], float scale_log2,
                                                float bias0, float bias1, SoftmaxState& st, float (&acc)[8][4]) {
    float ca[4] = {0.0f, 0.0f, 0.0f, 0.0f}, cb[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
    for (int c = 0; c < 8; ++c) {
        const int sh = 8 * (c & 1);
        const uint32_t wa = word_of(d0.ka, c >> 1) >> sh, wb = word_of(d0.kb, c >> 1) >> sh;
        mma_f16(ca, kq4_lo(wa), kq4_lo(wb), kq4_hi(wa), kq4_hi(wb), qf[2 * c], qf[2 * c + 1]);
        const uint32_t xa = word_of(d1.ka, c >> 1) >> sh, xb = word_of(d1.kb, c >> 1) >> sh;
        mma_f16(cb, kq4_lo(xa), kq4_lo(xb), kq4_hi(xa), kq4_hi(xb), qf[2 * c], qf[2 * c + 1]);
    }
    float pw[4];
    softmax_tile<false>(st, acc, ca, d0.fk * scale_log2, bias0, bias1, true, true, pw);
    uint32_t b0 = movmatrix_trans(pack_f16(pw[0] * d0.fv, pw[1] * d0.fv));
    uint32_t b1 = movmatrix_trans(pack_f16(pw[2] * d0.fv, pw[3] * d0.fv));
#pragma unroll
    for (int x = 0; x < 8; ++x) {
        const uint32_t w = word_of(x < 4 ? d0.va : d0.vb, x & 3);
        mma_f16(acc[x], dq4_lo(w), dq4_hi(w), dq4_lo(w >> 8), dq4_hi(w >> 8), b0, b1);
    }
    softmax_tile<false>(st, acc, cb, d1.fk * scale_log2, bias0, bias1, true, true, pw);
    b0 = movmatrix_trans(pack_f16(pw[0] * d1.fv, pw[1] * d1.fv));
    b1 = movmatrix_trans(pack_f16(pw[2] * d1.fv, pw[3] * d1.fv));
#pragma unroll
    for (int x = 0; x < 8; ++x) {
        const uint32_t w = word_of(x < 4 ? d1.va : d1.vb, x & 3);
        mma_f16(acc[x], dq4_lo(w), dq4_hi(w), dq4_lo(w >> 8), dq4_hi(w >> 8), b0, b1);
    }
}

// ---- INT8 cache (K8V8) ----------------------------------------------------------------------------------------
// A 16-row tile is 2 KB of K codes (row-major, 128 B per row) and 2 KB of V codes (operand order, see
// vq8_byte_offset).  K bytes enter Q.K^T as fp16 subnormals: byte ^ 0x80 = code + 128 in mantissa bits 0-7, upper byte
// zero, is (code + 128) * 2^-24; a byte permute builds two of them per register and the +128 becomes a per-head score
// constant.  V bytes are made exact: (byte ^ 0x80) under the constant byte 0x64 is fp16 1024 + code + 128, minus 1152.
struct QTile8 {
    uint4 k[4];          // row r: bytes [16j, +16) in k[0] and [64 + 16j, +16) in k[1]; row r + 8 in k[2], k[3]
    uint4 v[4];          // this lane's 16 bytes of each of the V tile's four 512-byte runs
    float fk, fv;
};

// FP8 e4m3 bytes: (byte & 0x7F) << 7 under the sign bit is the fp16 number with the same exponent and mantissa fields,
// i.e. the code's value times 2^-8 (exponent bias 15 against 7), subnormals included.  K leaves the 2^-8 to the score
// scale, V multiplies it back (exact: |code| <= 448).
__device__ __forceinline__ uint32_t e4m3_pair(uint32_t w, uint32_t sel) {     // sel: 0x1404 bytes 0,1; 0x3424 bytes 2,3
    const uint32_t x = __byte_perm(w, 0u, sel);                               // each byte in the high byte of its half
    const uint32_t mag = (x >> 1) & 0x3F803F80u;
    uint32_t h;
    asm("lop3.b32 %0, %1, 0x80008000, %2, 0xEA;" : "=r"(h) : "r"(x), "r"(mag));      // (x & sign bits) | mag
    return h;
}

template <bool RAGGED, bool FP8 = false>
__device__ __forceinline__ void quant_tile8(const QTile8& d, const uint32_t (&qf)[16], float scale_log2, float bias0, float bias1,
                                            int rows_valid, int r, SoftmaxState& st, float (&acc)[8][4]) {
    float c4[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
    for (int c = 0; c < 8; ++c) {
        if (FP8) {
            const uint32_t wa = word_of(d.k[c >> 2], c & 3), wb = word_of(d.k[2 + (c >> 2)], c & 3);
            mma_f16(c4, e4m3_pair(wa, 0x1404), e4m3_pair(wb, 0x1404), e4m3_pair(wa, 0x3424), e4m3_pair(wb, 0x3424),
                    qf[2 * c], qf[2 * c + 1]);
        } else {
            const uint32_t wa = word_of(d.k[c >> 2], c & 3) ^ 0x80808080u, wb = word_of(d.k[2 + (c >> 2)], c & 3) ^ 0x80808080u;
            mma_f16(c4, __byte_perm(wa, 0u, 0x4140), __byte_perm(wb, 0u, 0x4140), __byte_perm(wa, 0u, 0x4342),
                    __byte_perm(wb, 0u, 0x4342), qf[2 * c], qf[2 * c + 1]);
        }
    }
    float pw[4];
    softmax_tile<RAGGED>(st, acc, c4, d.fk * scale_log2, bias0, bias1, r < rows_valid, r + 8 < rows_valid, pw);
    const uint32_t b0 = movmatrix_trans(pack_f16(pw[0] * d.fv, pw[1] * d.fv));
    const uint32_t b1 = movmatrix_trans(pack_f16(pw[2] * d.fv, pw[3] * d.fv));
    auto exact = [](uint32_t w, uint32_t sel) {           // two bytes of w -> packed fp16 code values
        uint32_t h = __byte_perm(w, 0x64646464u, sel);
        asm("sub.rn.f16x2 %0, %1, %2;" : "=r"(h) : "r"(h), "r"(0x64806480u));
        return h;
    };
    auto value8 = [](uint32_t w, uint32_t sel) {          // two e4m3 bytes of w -> packed fp16 values
        uint32_t h = e4m3_pair(w, sel);
        asm("mul.rn.f16x2 %0, %1, %2;" : "=r"(h) : "r"(h), "r"(0x5C005C00u));         // times 256
        return h;
    };
#pragma unroll
    for (int x = 0; x < 8; ++x) {
        if (FP8) {
            const uint32_t w0 = word_of(d.v[x >> 1], 2 * (x & 1)), w1 = word_of(d.v[x >> 1], 2 * (x & 1) + 1);
            mma_f16(acc[x], value8(w0, 0x1404), value8(w0, 0x3424), value8(w1, 0x1404), value8(w1, 0x3424), b0, b1);
            continue;
        }
        const uint32_t w0 = word_of(d.v[x >> 1], 2 * (x & 1)) ^ 0x80808080u, w1 = word_of(d.v[x >> 1], 2 * (x & 1) + 1) ^ 0x80808080u;
        mma_f16(acc[x], exact(w0, 0x4140), exact(w0, 0x4342), exact(w1, 0x4140), exact(w1, 0x4342), b0, b1);
    }
}

template <int KVF>      // cache code format: HYQ_FMT_INT4, HYQ_FMT_INT8 or HYQ_FMT_FP8_E4M3
__global__ void __launch_bounds__(DEC_THREADS, DEC_CTAS_PER_SM)
decode_kernel(const DecParams p) {
    constexpr bool FMT8 = KVF != HYQ_FMT_INT4;             // byte-wide codes
    constexpr bool FP8 = KVF == HYQ_FMT_FP8_E4M3;
    const int split = blockIdx.x;
    // blockIdx.y = (b * Hkv + kv head) * hgroups + head group: up to 8 of the KV head's g query heads per CTA
    const long unit = blockIdx.y / p.hgroups;
    const int h_base = (int)(blockIdx.y % p.hgroups) * DEC_MAX_GROUP, g_here = min(DEC_MAX_GROUP, p.g - h_base);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, r = lane >> 2, j = lane & 3;
    // the merge kernel may be made resident while this grid runs (programmatic dependent launch): it waits for
    // this grid's completion before it reads anything, so only its launch latency is taken off the path
    asm volatile("griddepcontrol.launch_dependents;");

    __shared__ __align__(16) uint16_t qs[DEC_MAX_GROUP][HYQ_D];      // bf16 bits, heads >= g zero
    __shared__ float red_ml[DEC_WARPS][DEC_MAX_GROUP][2];
    __shared__ float q_sum[DEC_MAX_GROUP];                            // sum over channels of q as the K product sees it
    // per warp: a ring of DEC_STAGES tiles (1 KB of K codes + 1 KB of V codes each) filled by cp.async; every lane
    // reads back exactly the bytes it copied, so the ring needs no barrier.  Reused (after a CTA barrier) for the
    // warps' accumulators when the CTA merges them.
    extern __shared__ __align__(16) uint8_t ring_mem[];
    float (*red_acc)[DEC_MAX_GROUP][HYQ_D] = reinterpret_cast<float (*)[DEC_MAX_GROUP][HYQ_D]>(ring_mem);
    static_assert(DEC_STAGES * DEC_STAGE_BYTES >= DEC_MAX_GROUP * HYQ_D * 4, "rings too small for the merge");

    {   // q of the g heads of this KV head: thread t loads 8 channels of head t >> 4
        const int h = threadIdx.x >> 4, c8 = threadIdx.x & 15;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (h < g_here) v = __ldg(p.q + (unit * p.g + h_base + h) * 16 + c8);
        *reinterpret_cast<uint4*>(&qs[h][c8 * 8]) = v;
        // Odd channels sit in the high nibbles: their q enters the product as fp16(q / 16), times 16 here.
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
        float sum = 0.0f;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            sum += __half2float(__float2half_rn(bf16_lo(w[i])));
            sum += FMT8 ? __half2float(__float2half_rn(bf16_hi(w[i])))
                        : 16.0f * __half2float(__float2half_rn(bf16_hi(w[i]) * 0.0625f));
        }
#pragma unroll
        for (int o = 1; o < 16; o <<= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
        if (c8 == 0) q_sum[h] = sum;
    }
    __syncthreads();

    long nQ = p.nQ;
    int n_vl = p.k, n_win = p.W, n_stg = p.n_s;
    if (p.lens) {                                           // ragged batch: this sequence's own row counts
        // (clamped to the buffers' capacities: a bad length then shortens the walk instead of leaving the allocation)
        const int4 l = __ldg(p.lens + unit / p.Hkv);
        nQ = min(max((long)l.x, 0L), p.sQ); n_vl = min(max(l.y, 0), p.sK); n_win = min(max(l.z, 0), p.sW); n_stg = min(max(l.w, 0), p.Ws);
    }
    const long Tq = (nQ + 15) / 16;
    const int Tvl = (n_vl + 15) / 16, Ts = (n_stg + 15) / 16, Tw = (n_win + 15) / 16;
    // Every slice takes the same share of the INT4 tiles AND of the bf16 tiles (a bf16 tile moves four times the
    // bytes and goes through a different loop), so all CTAs of a head carry the same mix of work.
    const long Tf = Tvl + Ts + Tw;
    const long q_lo = Tq * split / p.splits, q_hi = Tq * (split + 1) / p.splits;
    const long f_lo = Tq + Tf * split / p.splits, f_hi = Tq + Tf * (split + 1) / p.splits;

    SoftmaxState st = {-INFINITY, -INFINITY, 0.0f, 0.0f};
    float acc[8][4];
#pragma unroll
    for (int x = 0; x < 8; ++x) acc[x][0] = acc[x][1] = acc[x][2] = acc[x][3] = 0.0f;

    // ---------------- quantized prefix ----------------
    if (!FMT8 && q_lo + warp < q_hi) {
        uint32_t qf[16];                                   // q^T operand, fp16: k-step c -> qf[2c], qf[2c+1]
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            const int base = 32 * j + 8 * (c >> 1) + 2 * (c & 1);
            const uint16_t* qr = qs[r];
            auto f16 = [&](int ch) { return __float2half_rn(__uint_as_float((uint32_t)qr[ch] << 16)); };
            const __half2 h0 = __halves2half2(f16(base), f16(base + 4));
#if DEC_K_SUBNORMAL
            auto f16s = [&](int ch) { return __float2half_rn(__uint_as_float((uint32_t)qr[ch] << 16) * 0.0625f); };
            const __half2 h1 = __halves2half2(f16s(base + 1), f16s(base + 5));
#else
            const __half2 h1 = __halves2half2(f16(base + 1), f16(base + 5));
#endif
            qf[2 * c] = *reinterpret_cast<const uint32_t*>(&h0);
            qf[2 * c + 1] = *reinterpret_cast<const uint32_t*>(&h1);
        }
        // this warp's tiles: t0, t0 + 4, ...  Tile i is copied into ring stage i % DEC_STAGES DEC_STAGES tiles ahead
        // of its use; one commit group per tile (empty past the end) keeps the group arithmetic uniform.
        const long t0 = q_lo + warp;
        const int n_my = (int)((q_hi - t0 + DEC_WARPS - 1) / DEC_WARPS);
        const bool has_ragged = (nQ & 15) && t0 + (long)(n_my - 1) * DEC_WARPS == Tq - 1;
        const uint8_t* gk = p.kq + unit * p.sQ * 64 + t0 * 1024 + lane * 16;
        const uint8_t* gv = p.vq + unit * (p.sQ / 16) * DEC_VTILE_BYTES + t0 * 1024 + lane * 16;
        const int gshift = p.gshift;
        const float* pks = p.ks + unit * (p.sQ >> (p.gshift + 4));
        const float* pvs = p.vs + unit * (p.sQ >> (p.gshift + 4));
        const uint32_t ring = (uint32_t)__cvta_generic_to_shared(ring_mem) + warp * (DEC_STAGES * DEC_STAGE_BYTES) + lane * 16;
        auto issue = [&](uint32_t stage_addr) {
            cp_async16(stage_addr, gk); cp_async16(stage_addr + 512, gk + 512);
            cp_async16(stage_addr + 1024, gv); cp_async16(stage_addr + 1536, gv + 512);
            gk += DEC_WARPS * 1024; gv += DEC_WARPS * 1024;
        };
#pragma unroll
        for (int s = 0; s < DEC_STAGES; ++s) {
            if (s < n_my) issue(ring + s * DEC_STAGE_BYTES);
            cp_async_commit();
        }
        uint32_t stage_addr = ring;
        const float kscale = p.scale_log2 * DEC_K_UNIT;
        const float b0 = DEC_K_SUBNORMAL ? q_sum[2 * j] * (8.0f / DEC_K_UNIT) : 0.0f;
        const float b1 = DEC_K_SUBNORMAL ? q_sum[2 * j + 1] * (8.0f / DEC_K_UNIT) : 0.0f;
        const int n_full = n_my - (has_ragged ? 1 : 0);
        auto fetch = [&](QTile& d, int i) {                 // ring stage of tile i -> registers, then refill it
            d.ka = lds128(stage_addr); d.kb = lds128(stage_addr + 512);
            d.va = lds128(stage_addr + 1024); d.vb = lds128(stage_addr + 1536);
            const int grp = ((int)t0 + i * DEC_WARPS) >> gshift;
            d.fk = __ldg(pks + grp); d.fv = __ldg(pvs + grp);
            if (i + DEC_STAGES < n_my) issue(stage_addr);   // own bytes only: no barrier
            cp_async_commit();
            stage_addr = (i % DEC_STAGES == DEC_STAGES - 1) ? ring : stage_addr + DEC_STAGE_BYTES;
        };
        int i = 0;
#if DEC_PAIR
        for (; i + 2 <= n_full; i += 2) {
            cp_async_wait<DEC_STAGES - 2>();                // tiles i and i + 1 have landed
            QTile A, B;
            fetch(A, i);
            fetch(B, i + 1);
            quant_tile_pair(A, B, qf, kscale, b0, b1, st, acc);
        }
#endif
        for (; i < n_my; ++i) {
            cp_async_wait<DEC_STAGES - 1>();                // tile i has landed
            QTile A;
            fetch(A, i);
            if (i >= n_full) quant_tile<true>(A, qf, kscale, b0, b1, (int)(nQ & 15), r, st, acc);
            else quant_tile<false>(A, qf, kscale, b0, b1, 16, r, st, acc);
        }
    }
    if (FMT8 && q_lo + warp < q_hi) {
        uint32_t qf[16];                                   // k-step c: channels 64 (c >> 2) + 16 j + 4 (c & 3) + {0,1} and + {2,3}
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            const int base = 64 * (c >> 2) + 16 * j + 4 * (c & 3);
            const uint16_t* qr = qs[r];
            auto f16 = [&](int ch) { return __float2half_rn(__uint_as_float((uint32_t)qr[ch] << 16)); };
            const __half2 h0 = __halves2half2(f16(base), f16(base + 1)), h1 = __halves2half2(f16(base + 2), f16(base + 3));
            qf[2 * c] = *reinterpret_cast<const uint32_t*>(&h0);
            qf[2 * c + 1] = *reinterpret_cast<const uint32_t*>(&h1);
        }
        constexpr int ST8 = 2, ST8_BYTES = DEC_STAGES * DEC_STAGE_BYTES / ST8;      // the same ring as two 4 KB stages
        static_assert(ST8_BYTES == 4096, "an INT8 tile is 2 KB of K and 2 KB of V");
        const long t0 = q_lo + warp;
        const int n_my = (int)((q_hi - t0 + DEC_WARPS - 1) / DEC_WARPS);
        const bool has_ragged = (nQ & 15) && t0 + (long)(n_my - 1) * DEC_WARPS == Tq - 1;
        const uint8_t* gk = p.kq + unit * p.sQ * 128 + t0 * 2048 + r * 128 + j * 16;       // bytes [16j, +16) and [64 + 16j, +16) of row r
        const uint8_t* gv = p.vq + unit * (p.sQ / 16) * 2048 + t0 * 2048 + lane * 16;
        const int gshift = p.gshift;
        const float* pks = p.ks + unit * (p.sQ >> (p.gshift + 4));
        const float* pvs = p.vs + unit * (p.sQ >> (p.gshift + 4));
        const uint32_t ring = (uint32_t)__cvta_generic_to_shared(ring_mem) + warp * (DEC_STAGES * DEC_STAGE_BYTES) + lane * 16;
        auto issue = [&](uint32_t sa) {
            cp_async16(sa, gk); cp_async16(sa + 512, gk + 64);
            cp_async16(sa + 1024, gk + 1024); cp_async16(sa + 1536, gk + 1088);
#pragma unroll
            for (int i = 0; i < 4; ++i) cp_async16(sa + 2048 + i * 512, gv + i * 512);
            gk += DEC_WARPS * 2048; gv += DEC_WARPS * 2048;
        };
#pragma unroll
        for (int s = 0; s < ST8; ++s) {
            if (s < n_my) issue(ring + s * ST8_BYTES);
            cp_async_commit();
        }
        // INT8: subnormal operand (2^-24) and the +128 offset; FP8: the 2^-8 of the exponent-bias trick, no offset
        const float kscale = p.scale_log2 * (FP8 ? 256.0f : 16777216.0f);
        const float b0 = FP8 ? 0.0f : q_sum[2 * j] * (128.0f / 16777216.0f), b1 = FP8 ? 0.0f : q_sum[2 * j + 1] * (128.0f / 16777216.0f);
        for (int i = 0; i < n_my; ++i) {
            cp_async_wait<ST8 - 1>();                       // tile i has landed
            const uint32_t sa = ring + (i & 1) * ST8_BYTES;
            QTile8 A;
#pragma unroll
            for (int u = 0; u < 4; ++u) { A.k[u] = lds128(sa + u * 512); A.v[u] = lds128(sa + 2048 + u * 512); }
            const int grp = ((int)t0 + i * DEC_WARPS) >> gshift;
            A.fk = __ldg(pks + grp); A.fv = __ldg(pvs + grp);
            if (i + ST8 < n_my) issue(sa);                  // own bytes only: no barrier
            cp_async_commit();
            if (has_ragged && i == n_my - 1) quant_tile8<true, FP8>(A, qf, kscale, b0, b1, (int)(nQ & 15), r, st, acc);
            else quant_tile8<false, FP8>(A, qf, kscale, b0, b1, 16, r, st, acc);
        }
    }
    cp_async_wait<0>();

    // ---------------- bf16 segments: vertical rows, staging, window ----------------
    // continue the round-robin where the INT4 tiles left off so that the warps stay balanced
    long t = f_lo + ((warp - (q_hi - q_lo)) % DEC_WARPS + DEC_WARPS) % DEC_WARPS;
    if (t < f_hi) {
        uint32_t qb[16];                                   // q^T operand, bf16
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            const int base = 32 * (c >> 1) + 8 * j + 4 * (c & 1);
            qb[2 * c] = *reinterpret_cast<const uint32_t*>(&qs[r][base]);
            qb[2 * c + 1] = *reinterpret_cast<const uint32_t*>(&qs[r][base + 2]);
        }
        for (; t < f_hi; t += DEC_WARPS) {
            long u = t - Tq;
            const uint4 *kseg, *vseg;
            int n;
            if (u < Tvl) { kseg = p.k_vl + unit * p.sK * 16; vseg = p.v_vl + unit * p.sK * 16; n = n_vl; }
            else if ((u -= Tvl) < Ts) { kseg = p.k_s + unit * p.Ws * 16; vseg = p.v_s + unit * p.Ws * 16; n = n_stg; }
            else { u -= Ts; kseg = p.k_win + unit * p.sW * 16; vseg = p.v_win + unit * p.sW * 16; n = n_win; }
            const int row0 = (int)u * 16;
            const int ra = min(row0 + r, n - 1), rb = min(row0 + r + 8, n - 1);
            uint4 ka[4], kb[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) { ka[i] = __ldg(kseg + (long)ra * 16 + 4 * i + j); kb[i] = __ldg(kseg + (long)rb * 16 + 4 * i + j); }
            float c4[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const int wd = 2 * (c & 1);
                mma_bf16(c4, word_of(ka[c >> 1], wd), word_of(kb[c >> 1], wd), word_of(ka[c >> 1], wd + 1),
                         word_of(kb[c >> 1], wd + 1), qb[2 * c], qb[2 * c + 1]);
            }
            uint4 vv[4][2];
#pragma unroll
            for (int sIdx = 0; sIdx < 4; ++sIdx) {
                const int key = min(row0 + 2 * j + (sIdx & 1) + 8 * (sIdx >> 1), n - 1);
                vv[sIdx][0] = __ldg(vseg + (long)key * 16 + r);
                vv[sIdx][1] = __ldg(vseg + (long)key * 16 + 8 + r);
            }
            float pw[4];
            if (row0 + 16 > n) softmax_tile<true>(st, acc, c4, p.scale_log2, 0.0f, 0.0f, row0 + r < n, row0 + r + 8 < n, pw);
            else softmax_tile<false>(st, acc, c4, p.scale_log2, 0.0f, 0.0f, true, true, pw);
            // The weights go into the bf16 product as a sum of two bf16 numbers (p = hi + lo, 16 significant bits):
            // with one bf16 the 2^-9 rounding of a dominant full-precision key would show in the output.
            const uint32_t h01 = pack_bf16(pw[0], pw[1]), h23 = pack_bf16(pw[2], pw[3]);
            const uint32_t l01 = pack_bf16(pw[0] - bf16_lo(h01), pw[1] - bf16_hi(h01));
            const uint32_t l23 = pack_bf16(pw[2] - bf16_lo(h23), pw[3] - bf16_hi(h23));
            const uint32_t b0 = movmatrix_trans(h01), b1 = movmatrix_trans(h23);
            const uint32_t b0l = movmatrix_trans(l01), b1l = movmatrix_trans(l23);
#pragma unroll
            for (int x = 0; x < 8; ++x) {
                const uint32_t w0 = word_of(vv[0][x >> 2], x & 3), w1 = word_of(vv[1][x >> 2], x & 3);
                const uint32_t w2 = word_of(vv[2][x >> 2], x & 3), w3 = word_of(vv[3][x >> 2], x & 3);
                const uint32_t a0 = __byte_perm(w0, w1, 0x5410), a1 = __byte_perm(w0, w1, 0x7632);
                const uint32_t a2 = __byte_perm(w2, w3, 0x5410), a3 = __byte_perm(w2, w3, 0x7632);
                mma_bf16(acc[x], a0, a1, a2, a3, b0, b1);
                mma_bf16(acc[x], a0, a1, a2, a3, b0l, b1l);
            }
        }
    }

    // ---------------- merge the warps' states, write the slice's partial result ----------------
    __syncthreads();                                       // every warp is done with its ring
#pragma unroll
    for (int o = 4; o < 32; o <<= 1) {
        st.l0 += __shfl_xor_sync(0xffffffffu, st.l0, o);
        st.l1 += __shfl_xor_sync(0xffffffffu, st.l1, o);
    }
    if (r == 0) {
        red_ml[warp][2 * j][0] = st.m0; red_ml[warp][2 * j][1] = st.l0;
        red_ml[warp][2 * j + 1][0] = st.m1; red_ml[warp][2 * j + 1][1] = st.l1;
    }
#pragma unroll
    for (int x = 0; x < 8; ++x) {
        red_acc[warp][2 * j][acc_channel(x, r, 0)] = acc[x][0];
        red_acc[warp][2 * j + 1][acc_channel(x, r, 0)] = acc[x][1];
        red_acc[warp][2 * j][acc_channel(x, r, 1)] = acc[x][2];
        red_acc[warp][2 * j + 1][acc_channel(x, r, 1)] = acc[x][3];
    }
    __syncthreads();
    const long slot = (long)blockIdx.y * p.splits + split;
    for (int h = 0; h < g_here; ++h) {
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < DEC_WARPS; ++w) M = fmaxf(M, red_ml[w][h][0]);
        float L = 0.0f, A = 0.0f;
#pragma unroll
        for (int w = 0; w < DEC_WARPS; ++w) {
            const float mw = red_ml[w][h][0];
            const float wt = mw == -INFINITY ? 0.0f : ex2(mw - M);
            L += red_ml[w][h][1] * wt;
            A += red_acc[w][h][threadIdx.x] * wt;
        }
        p.part_acc[(slot * DEC_MAX_GROUP + h) * HYQ_D + threadIdx.x] = A;
        if (threadIdx.x == 0) {
            p.part_ml[(slot * DEC_MAX_GROUP + h) * 2] = M;
            p.part_ml[(slot * DEC_MAX_GROUP + h) * 2 + 1] = L;
        }
    }
}

// ReduceSoftmax of Algorithm 3 over the slices; one CTA per (b, kv head, query head), one thread per channel.
// The slices' (m, l) pairs are staged in shared memory first so that the channel loop is a run of
// independent loads (the kernel is pure latency otherwise: it moves a few hundred KB).
constexpr int DEC_MAX_SPLITS = 1024;
__global__ void __launch_bounds__(HYQ_D)
decode_merge_kernel(const float* __restrict__ part_acc, const float* __restrict__ part_ml, int g, int hgroups, int splits,
                    int out_fp32, void* __restrict__ out, float* __restrict__ lse) {
    const long unit = blockIdx.x;                                  // (b * Hkv + kv head) * hgroups + head group
    const int h = blockIdx.y;                                      // head within the group
    const int h_base = (int)(unit % hgroups) * DEC_MAX_GROUP;
    if (h_base + h >= g) return;
    asm volatile("griddepcontrol.wait;" ::: "memory");       // the slice kernel has completed and its results are visible
    __shared__ float wt[DEC_MAX_SPLITS];
    __shared__ float red[2][HYQ_D / 32];
    const long slot0 = unit * splits * DEC_MAX_GROUP + h;          // slice s sits at slot0 + s * DEC_MAX_GROUP
    float M = -INFINITY;
    for (int s = threadIdx.x; s < splits; s += HYQ_D) {
        wt[s] = __ldg(part_ml + (slot0 + (long)s * DEC_MAX_GROUP) * 2);
        M = fmaxf(M, wt[s]);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
    if ((threadIdx.x & 31) == 0) red[0][threadIdx.x >> 5] = M;
    __syncthreads();
    M = fmaxf(fmaxf(red[0][0], red[0][1]), fmaxf(red[0][2], red[0][3]));
    float L = 0.0f;
    for (int s = threadIdx.x; s < splits; s += HYQ_D) {
        const float w = wt[s] == -INFINITY ? 0.0f : ex2(wt[s] - M);
        L += __ldg(part_ml + (slot0 + (long)s * DEC_MAX_GROUP) * 2 + 1) * w;
        wt[s] = w;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) L += __shfl_xor_sync(0xffffffffu, L, o);
    if ((threadIdx.x & 31) == 0) red[1][threadIdx.x >> 5] = L;
    __syncthreads();
    L = (red[1][0] + red[1][1]) + (red[1][2] + red[1][3]);
    float A = 0.0f;
#pragma unroll 8
    for (int s = 0; s < splits; ++s) A += __ldg(part_acc + (slot0 + (long)s * DEC_MAX_GROUP) * HYQ_D + threadIdx.x) * wt[s];
    const float o = L > 0.0f ? A / L : 0.0f;               // a sequence with no cached row at all: zeros
    const long head = (unit / hgroups) * g + h_base + h;
    const long oi = head * HYQ_D + threadIdx.x;
    if (out_fp32) static_cast<float*>(out)[oi] = o;
    else static_cast<__nv_bfloat16*>(out)[oi] = __float2bfloat16_rn(o);
    if (lse && threadIdx.x == 0) lse[head] = (M + log2f(L)) * 0.6931471805599453f;
}

static long decode_tiles(const hyq_kv_cache& c) {
    const CacheGeo g = cache_geo(c);
    return (g.nQ + 15) / 16 + (c.k + 15) / 16 + (c.n_staging + 15) / 16 + (g.W + 15) / 16;
}

int decode_auto_splits(const hyq_kv_cache& c) {
    const long units = (long)c.B * c.Hkv * ((c.Hq / c.Hkv + DEC_MAX_GROUP - 1) / DEC_MAX_GROUP);
    const long T = decode_tiles(c);
    long s = 148L * DEC_CTAS_PER_SM / units;            // one full wave of resident CTAs, never a second partial one
    // Few heads (small batches) cannot fill the wave with slices long enough to pay for a CTA's prologue, its partial
    // results and their merge: aim at 64 tiles per slice (measured at batch 1: 32 slices 20.4 us, 64 slices 22.6 us),
    // but keep at least 8 slices of two tiles per warp for short caches.
    const long cap = T / 8 > 1 ? T / 8 : 1;
    const long floor_s = cap < 8 ? cap : 8;
    long want = T / 64;
    if (want < floor_s) want = floor_s;
    if (s > want) s = want;
    if (s > 64) s = 64;
    return (int)(s < 1 ? 1 : s);
}

size_t decode_workspace_bytes(const hyq_kv_cache& c, int splits) {
    const size_t slots = (size_t)c.B * c.Hkv * ((c.Hq / c.Hkv + DEC_MAX_GROUP - 1) / DEC_MAX_GROUP) * splits * DEC_MAX_GROUP;
    return align_up(slots * HYQ_D * sizeof(float), 16) + align_up(slots * 2 * sizeof(float), 16);
}

int launch_decode(const void* q, const hyq_kv_cache& c, const int32_t* lengths, float alpha, int splits, int out_dtype,
                  void* out, float* lse, void* workspace, cudaStream_t st) {
    const CacheGeo geo = cache_geo(c);
    DecParams p;
    p.g = c.Hq / c.Hkv; p.splits = splits;
    p.hgroups = (p.g + DEC_MAX_GROUP - 1) / DEC_MAX_GROUP;
    const long units = (long)c.B * c.Hkv * p.hgroups;         // CTA rows of the grid: (b, kv head, head group)
    p.gshift = c.group == 32 ? 1 : c.group == 64 ? 2 : 3;
    p.Hkv = c.Hkv; p.lens = reinterpret_cast<const int4*>(lengths);
    p.nQ = geo.nQ; p.sQ = geo.sQ; p.k = c.k; p.W = geo.W; p.n_s = c.n_staging;
    p.sK = (int)geo.sK; p.sW = (int)geo.sW; p.Ws = c.staging_capacity;
    p.scale_log2 = alpha * 1.4426950408889634f;
    p.kq = static_cast<const uint8_t*>(c.kq_codes); p.vq = static_cast<const uint8_t*>(c.vq_codes);
    p.ks = c.kq_scales; p.vs = c.vq_scales;
    p.k_vl = static_cast<const uint4*>(c.k_vl); p.v_vl = static_cast<const uint4*>(c.v_vl);
    p.k_s = static_cast<const uint4*>(c.k_s); p.v_s = static_cast<const uint4*>(c.v_s);
    p.k_win = static_cast<const uint4*>(c.k_win); p.v_win = static_cast<const uint4*>(c.v_win);
    p.q = static_cast<const uint4*>(q);
    const size_t slots = (size_t)units * splits * DEC_MAX_GROUP;
    p.part_acc = static_cast<float*>(workspace);
    p.part_ml = reinterpret_cast<float*>(static_cast<char*>(workspace) + align_up(slots * HYQ_D * sizeof(float), 16));
    constexpr int ring_bytes = DEC_WARPS * DEC_STAGES * DEC_STAGE_BYTES;
    // the opt-in to more than 48 KB of dynamic shared memory is per device: once per device and process
    // (same value every time, so a race between host threads is benign)
    static bool attr_set[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return HYQ_ERR_CUDA;
    if (!attr_set[dev]) {
        if (cudaFuncSetAttribute(decode_kernel<HYQ_FMT_INT4>, cudaFuncAttributeMaxDynamicSharedMemorySize, ring_bytes) != cudaSuccess ||
            cudaFuncSetAttribute(decode_kernel<HYQ_FMT_INT8>, cudaFuncAttributeMaxDynamicSharedMemorySize, ring_bytes) != cudaSuccess ||
            cudaFuncSetAttribute(decode_kernel<HYQ_FMT_FP8_E4M3>, cudaFuncAttributeMaxDynamicSharedMemorySize, ring_bytes) != cudaSuccess)
            return HYQ_ERR_CUDA;
        attr_set[dev] = true;
    }
    const dim3 grid((unsigned)splits, (unsigned)units);
    if (c.format == HYQ_FMT_INT8) decode_kernel<HYQ_FMT_INT8><<<grid, DEC_THREADS, ring_bytes, st>>>(p);
    else if (c.format == HYQ_FMT_FP8_E4M3) decode_kernel<HYQ_FMT_FP8_E4M3><<<grid, DEC_THREADS, ring_bytes, st>>>(p);
    else decode_kernel<HYQ_FMT_INT4><<<grid, DEC_THREADS, ring_bytes, st>>>(p);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)units, (unsigned)(p.g < DEC_MAX_GROUP ? p.g : DEC_MAX_GROUP));
    cfg.blockDim = dim3(HYQ_D);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const float* pa = p.part_acc;
    const float* pm = p.part_ml;
    if (cudaLaunchKernelEx(&cfg, decode_merge_kernel, pa, pm, p.g, p.hgroups, splits, out_dtype, out, lse) != cudaSuccess) return HYQ_ERR_CUDA;
    return launch_status();
}

}  // namespace hyq
