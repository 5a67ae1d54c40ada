// Column-mass vertical-line selector (Eq. 4-5): S(p) = sum over a set of tail queries of their softmax
// probability on key p, then top-k over the non-window prefix.
//
// The scores decide an index set that has to match the reference bit for bit, so the arithmetic is fixed
// operation by operation, all fp64 with explicit round-to-nearest intrinsics (no contraction):
//   s       = (fma chain over channels 0..127 from 0) * alpha
//   exp     = exp_det: two-part reduction by ln 2, degree-13 Taylor polynomial by Horner fma, exact 2^n scaling
//   row sum = per chunk of 64 keys: m_c = max, z_c = pairwise tree over exp(s - m_c) (the xor butterfly of a warp
//             IS that tree, the two warps of a CTA are its last level); then m = max m_c and
//             Z = sum_c z_c * exp(m_c - m) in ascending chunk order
//   S(p)    = sum over the queries in ascending order of exp(s - m_t) / Z_t
// Three kernels: chunk statistics (one pass over Q.K^T), their combination per query row, column sums (a second
// pass over the prefix columns); then the radix top-k of the Algorithm-1 selector.  Work is n_queries * L * 128
// fp64 fma per head and pass - a pre-pass for a handful of tail queries, not a second attention.
//
// Both passes use the same tile: a CTA of 256 threads owns 256 consecutive keys (four chunks) of one (b, kv head), each thread
// keeps its key row in registers as bf16 pairs and scores it against MASS_TQ queries at a time, whose rows sit
// in shared memory as doubles (broadcast reads).
#include "common.cuh"

namespace hyq {

constexpr int MASS_KEYS = 64;        // keys per chunk of the row-sum definition (two warps)
constexpr int MASS_CHUNKS = 4;       // chunks per CTA (they share the staged query rows)
constexpr int MASS_THREADS = MASS_KEYS * MASS_CHUNKS;
#ifndef MASS_MIN_CTAS
#define MASS_MIN_CTAS 2                 // 128 registers: a few spilled words, twice the warps (measured 20 % faster)
#endif
constexpr int MASS_TQ = 8;           // queries scored together (independent fma chains per thread)
constexpr int MASS_QTILE = 64;       // query rows staged in shared memory at a time (64 KB of doubles)

__device__ __forceinline__ double exp_det(double x) {
    if (!(x >= -690.0)) return 0.0;
    const double n = rint(__dmul_rn(x, 1.4426950408889634));
    double r = __fma_rn(n, -6.93147180369123816490e-01, x);
    r = __fma_rn(n, -1.90821492927058770002e-10, r);
    double p = 1.0 / 6227020800.0;
    p = __fma_rn(p, r, 1.0 / 479001600.0);
    p = __fma_rn(p, r, 1.0 / 39916800.0);
    p = __fma_rn(p, r, 1.0 / 3628800.0);
    p = __fma_rn(p, r, 1.0 / 362880.0);
    p = __fma_rn(p, r, 1.0 / 40320.0);
    p = __fma_rn(p, r, 1.0 / 5040.0);
    p = __fma_rn(p, r, 1.0 / 720.0);
    p = __fma_rn(p, r, 1.0 / 120.0);
    p = __fma_rn(p, r, 1.0 / 24.0);
    p = __fma_rn(p, r, 1.0 / 6.0);
    p = __fma_rn(p, r, 0.5);
    p = __fma_rn(p, r, 1.0);
    p = __fma_rn(p, r, 1.0);
    return __dmul_rn(p, __longlong_as_double(((long long)n + 1023) << 52));
}

// this thread's key row (64 words of two bf16) -> registers; rows past the end read row `last`
__device__ __forceinline__ void load_key_row(const __nv_bfloat16* kh, int j, int last, uint32_t (&kw)[HYQ_D / 2]) {
    const uint4* src = reinterpret_cast<const uint4*>(kh + (long)min(j, last) * HYQ_D);
#pragma unroll
    for (int v = 0; v < HYQ_D / 8; ++v) {
        const uint4 w = __ldg(src + v);
        kw[4 * v] = w.x; kw[4 * v + 1] = w.y; kw[4 * v + 2] = w.z; kw[4 * v + 3] = w.w;
    }
}

// q rows [t0, t0 + n) of one head -> shared memory as doubles
__device__ __forceinline__ void stage_queries(const __nv_bfloat16* qrows, int n, double* qd) {
    for (int e = threadIdx.x; e < n * HYQ_D; e += MASS_THREADS) qd[e] = (double)__bfloat162float(qrows[e]);
}

// scores of this thread's key against MASS_TQ staged query rows: independent fma chains in channel order
__device__ __forceinline__ void score_queries(const uint32_t (&kw)[HYQ_D / 2], const double* qd, double alpha,
                                              double (&s)[MASS_TQ]) {
#pragma unroll
    for (int c = 0; c < MASS_TQ; ++c) s[c] = 0.0;
#pragma unroll
    for (int w = 0; w < HYQ_D / 2; ++w) {
        const double k0 = (double)bf16_lo(kw[w]), k1 = (double)bf16_hi(kw[w]);
#pragma unroll
        for (int c = 0; c < MASS_TQ; ++c) {
            const double2 qv = *reinterpret_cast<const double2*>(qd + c * HYQ_D + 2 * w);
            s[c] = __fma_rn(qv.x, k0, s[c]);
            s[c] = __fma_rn(qv.y, k1, s[c]);
        }
    }
#pragma unroll
    for (int c = 0; c < MASS_TQ; ++c) s[c] = __dmul_rn(s[c], alpha);
}

// Pass 1: per (query row, chunk) the chunk maximum and the tree sum of exp(s - max).
__global__ void __launch_bounds__(MASS_THREADS, MASS_MIN_CTAS)
mass_chunk_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ kmat, int Hq, int Hkv, int Lq,
                  int Lk, int nT, int n_chunks, double alpha, double* __restrict__ chunk_m, double* __restrict__ chunk_z) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    double* qd = reinterpret_cast<double*>(smem_raw);                 // [MASS_QTILE][D]
    __shared__ double red_m_all[MASS_CHUNKS][2][MASS_TQ], red_z_all[MASS_CHUNKS][2][MASS_TQ];
    const int cl = threadIdx.x / MASS_KEYS, tc = threadIdx.x % MASS_KEYS;   // chunk within the CTA, key within the chunk
    double (*red_m)[MASS_TQ] = red_m_all[cl];
    double (*red_z)[MASS_TQ] = red_z_all[cl];
    const int chunk = blockIdx.x * MASS_CHUNKS + cl, kvh = blockIdx.y, b = blockIdx.z, g = Hq / Hkv;
    const int j = chunk * MASS_KEYS + tc;
    const int lane = threadIdx.x & 31, wid = (threadIdx.x >> 5) & 1;
    uint32_t kw[HYQ_D / 2];
    load_key_row(kmat + ((long)b * Hkv + kvh) * Lk * HYQ_D, j, Lk - 1, kw);
    const int pos0 = Lk - nT;                                          // position of the first query of the set
    for (int r = 0; r < g; ++r) {
        const long bh = (long)b * Hq + (long)kvh * g + r;
        const __nv_bfloat16* qhead = q + (bh * Lq + (Lq - nT)) * HYQ_D;
        for (int t0 = 0; t0 < nT; t0 += MASS_QTILE) {
            const int nt = min(MASS_QTILE, nT - t0);
            const int nt_pad = (nt + MASS_TQ - 1) / MASS_TQ * MASS_TQ;
            __syncthreads();
            stage_queries(qhead + (long)t0 * HYQ_D, nt, qd);
            for (int e = nt * HYQ_D + threadIdx.x; e < nt_pad * HYQ_D; e += MASS_THREADS) qd[e] = 0.0;
            __syncthreads();
            for (int tq = 0; tq < nt; tq += MASS_TQ) {
                double s[MASS_TQ], m[MASS_TQ], z[MASS_TQ];
                score_queries(kw, qd + tq * HYQ_D, alpha, s);
#pragma unroll
                for (int c = 0; c < MASS_TQ; ++c) {
                    if (j > pos0 + t0 + tq + c) s[c] = -INFINITY;      // causal: key not visible to this query
                    m[c] = s[c];
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) m[c] = fmax(m[c], __shfl_xor_sync(0xffffffffu, m[c], o));
                }
                if (lane == 0) {
#pragma unroll
                    for (int c = 0; c < MASS_TQ; ++c) red_m[wid][c] = m[c];
                }
                __syncthreads();
#pragma unroll
                for (int c = 0; c < MASS_TQ; ++c) {
                    m[c] = fmax(red_m[0][c], red_m[1][c]);
                    z[c] = s[c] == -INFINITY ? 0.0 : exp_det(__dsub_rn(s[c], m[c]));
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) z[c] = __dadd_rn(z[c], __shfl_xor_sync(0xffffffffu, z[c], o));
                }
                if (lane == 0) {
#pragma unroll
                    for (int c = 0; c < MASS_TQ; ++c) red_z[wid][c] = z[c];
                }
                __syncthreads();
                if (tc < MASS_TQ && tq + tc < nt && chunk < n_chunks) {
                    const int c = tc;
                    const long slot = (bh * nT + t0 + tq + c) * n_chunks + chunk;
                    chunk_m[slot] = fmax(red_m[0][c], red_m[1][c]);
                    chunk_z[slot] = __dadd_rn(red_z[0][c], red_z[1][c]);
                }
                __syncthreads();                                       // red_m / red_z are rewritten by the next group
            }
        }
    }
}

// Row maximum and row sum from the chunk statistics: one thread per (b, h, query), chunks in ascending order.
__global__ void mass_combine_kernel(const double* __restrict__ chunk_m, const double* __restrict__ chunk_z, long rows,
                                    int nT, int Lk, int n_chunks, double* __restrict__ row_mz) {
    const long row = (long)blockIdx.x * blockDim.x + threadIdx.x;      // (bh * nT + t)
    if (row >= rows) return;
    const int t = (int)(row % nT);
    const int nc = (Lk - nT + t) / MASS_KEYS + 1;                      // chunks that hold a visible key
    const double* cm = chunk_m + row * n_chunks;
    const double* cz = chunk_z + row * n_chunks;
    double m = -INFINITY;
    for (int c = 0; c < nc; ++c) m = fmax(m, cm[c]);
    double Z = 0.0;
    for (int c = 0; c < nc; ++c) Z = __dadd_rn(Z, __dmul_rn(cz[c], exp_det(__dsub_rn(cm[c], m))));
    row_mz[2 * row] = m;
    row_mz[2 * row + 1] = Z;
}

// Pass 2: S(p) for the prefix keys, queries in ascending order.
__global__ void __launch_bounds__(MASS_THREADS, MASS_MIN_CTAS)
mass_column_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ kmat, int Hq, int Hkv, int Lq,
                   int Lk, int P, int nT, double alpha, const double* __restrict__ row_mz, double* __restrict__ scores) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    double* qd = reinterpret_cast<double*>(smem_raw);                 // [MASS_QTILE][D]
    __shared__ double mz[MASS_QTILE][2];
    const int kvh = blockIdx.y, b = blockIdx.z, g = Hq / Hkv;
    const int p = blockIdx.x * MASS_THREADS + threadIdx.x;
    uint32_t kw[HYQ_D / 2];
    load_key_row(kmat + ((long)b * Hkv + kvh) * Lk * HYQ_D, p, P - 1, kw);
    for (int r = 0; r < g; ++r) {
        const long bh = (long)b * Hq + (long)kvh * g + r;
        const __nv_bfloat16* qhead = q + (bh * Lq + (Lq - nT)) * HYQ_D;
        double S = 0.0;
        for (int t0 = 0; t0 < nT; t0 += MASS_QTILE) {
            const int nt = min(MASS_QTILE, nT - t0);
            const int nt_pad = (nt + MASS_TQ - 1) / MASS_TQ * MASS_TQ;
            __syncthreads();
            stage_queries(qhead + (long)t0 * HYQ_D, nt, qd);
            for (int e = nt * HYQ_D + threadIdx.x; e < nt_pad * HYQ_D; e += MASS_THREADS) qd[e] = 0.0;
            if (threadIdx.x < nt) {
                mz[threadIdx.x][0] = row_mz[2 * (bh * nT + t0 + threadIdx.x)];
                mz[threadIdx.x][1] = row_mz[2 * (bh * nT + t0 + threadIdx.x) + 1];
            }
            __syncthreads();
            for (int tq = 0; tq < nt; tq += MASS_TQ) {
                double s[MASS_TQ];
                score_queries(kw, qd + tq * HYQ_D, alpha, s);
#pragma unroll
                for (int c = 0; c < MASS_TQ; ++c)
                    if (tq + c < nt) S = __dadd_rn(S, __ddiv_rn(exp_det(__dsub_rn(s[c], mz[tq + c][0])), mz[tq + c][1]));
            }
        }
        if (p < P) scores[bh * P + p] = S;
    }
}

size_t select_mass_workspace_bytes(int B, int Hq, int Lk, int window, int n_queries) {
    const long P = (Lk - window > 0) ? Lk - window : 0;
    const long rows = (long)B * Hq * n_queries, n_chunks = (Lk + MASS_KEYS - 1) / MASS_KEYS;
    return align_up((size_t)B * Hq * P * sizeof(double), 256) + 2 * align_up((size_t)rows * n_chunks * sizeof(double), 256) +
           align_up((size_t)rows * 2 * sizeof(double), 256);
}

int launch_select_mass(const void* q, const void* k, int B, int Hq, int Hkv, int Lq, int Lk, int window, int n_queries,
                       int k_sel, double alpha, int32_t* idx_out, void* ws, cudaStream_t st) {
    const int P = Lk - window, nT = n_queries;
    const long rows = (long)B * Hq * nT;
    const int n_chunks = (Lk + MASS_KEYS - 1) / MASS_KEYS;
    char* base = static_cast<char*>(ws);
    double* scores = reinterpret_cast<double*>(base);
    base += align_up((size_t)B * Hq * P * sizeof(double), 256);
    double* chunk_m = reinterpret_cast<double*>(base);
    base += align_up((size_t)rows * n_chunks * sizeof(double), 256);
    double* chunk_z = reinterpret_cast<double*>(base);
    base += align_up((size_t)rows * n_chunks * sizeof(double), 256);
    double* row_mz = reinterpret_cast<double*>(base);
    const auto* qb = static_cast<const __nv_bfloat16*>(q);
    const auto* kb = static_cast<const __nv_bfloat16*>(k);

    constexpr int smem = MASS_QTILE * HYQ_D * (int)sizeof(double);     // 64 KB
    // (per device and process; same values every time, so a race between host threads is benign)
    static bool attr_set[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return HYQ_ERR_CUDA;
    if (!attr_set[dev]) {
        if (cudaFuncSetAttribute(mass_chunk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess ||
            cudaFuncSetAttribute(mass_column_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
            return HYQ_ERR_CUDA;
        attr_set[dev] = true;
    }
    mass_chunk_kernel<<<dim3((n_chunks + MASS_CHUNKS - 1) / MASS_CHUNKS, Hkv, B), MASS_THREADS, smem, st>>>(qb, kb, Hq, Hkv, Lq, Lk, nT, n_chunks, alpha, chunk_m, chunk_z);
    if (launch_status() != HYQ_OK) return HYQ_ERR_CUDA;
    mass_combine_kernel<<<(unsigned)((rows + 127) / 128), 128, 0, st>>>(chunk_m, chunk_z, rows, nT, Lk, n_chunks, row_mz);
    if (launch_status() != HYQ_OK) return HYQ_ERR_CUDA;
    mass_column_kernel<<<dim3((P + MASS_THREADS - 1) / MASS_THREADS, Hkv, B), MASS_THREADS, smem, st>>>(qb, kb, Hq, Hkv, Lq, Lk, P, nT, alpha,
                                                                                                row_mz, scores);
    if (launch_status() != HYQ_OK) return HYQ_ERR_CUDA;
    return launch_topk(scores, (long)B * Hq, P, k_sel, idx_out, st);
}

}  // namespace hyq
