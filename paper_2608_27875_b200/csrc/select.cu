// Vertical token identification (Algorithm 1): tail-query mean -> GQA-native dot-product
// scores over the non-window prefix -> exact top-k per query head.
//
// Three kernels, all bound by memory traffic:
//   tail_mean_kernel   qbar[b,h,:] = (1/t) sum of the last t query rows, fp64, added in row order
//   vscore_kernel      S[b,h,p] = qbar[b,h,:] . K[b,h/g,p,:], an fp64 fma chain in channel
//                      order; each K row is read once per KV head and scored for its g query heads
//   topk_kernel        per (b,h): MSB-first radix select of the k-th largest score on an
//                      order-preserving 64-bit key, then an ordered compaction that emits the
//                      selected positions ascending; equal scores go to the lower position.
// The fp64 chain is what makes the selected set reproducible bit for bit: ranking in lower
// precision flips pairs whose scores differ by less than its rounding error.
#include <mutex>

#include "common.cuh"

namespace hyq {

constexpr int SCORE_KEYS = 128;      // keys per CTA in vscore_kernel
constexpr int SCORE_GC = 4;          // query heads scored per pass over the staged K tile
constexpr int TOPK_THREADS = 1024;
constexpr int SCAN_DEPTH = 8;         // loads of the score row a thread of the radix select keeps in flight
constexpr int TOPK_CAND = 1536;      // candidate keys that the radix select keeps in shared memory

// -------------------------------------------------------------------------------------------
// The t tail rows are added in ascending row order in fp64, one running sum per (b, h, channel) - the order of
// Algorithm 1's mean as it is written down, so the result is the same double for every finite input, whatever the
// spread of the exponents (a split into partial sums would only agree while every partial sum is exact).  A CTA owns
// 32 channels of one (b, h): all its threads stage 512 rows at a time in shared memory (the loads are what takes
// time), then one thread per channel runs the addition chain over the staged rows.
constexpr int MEAN_CH = 32, MEAN_ROWS = 512, MEAN_THREADS = 256;

__global__ void __launch_bounds__(MEAN_THREADS)
tail_mean_kernel(const __nv_bfloat16* __restrict__ q, int Lq, int t, double* __restrict__ qbar) {
    __shared__ __nv_bfloat16 tile[MEAN_ROWS][MEAN_CH + 2];         // +2: the chain's column reads stay conflict-free enough
    const long bh = blockIdx.x;
    const int c0 = blockIdx.y * MEAN_CH;
    const __nv_bfloat16* base = q + (bh * Lq + (Lq - t)) * (long)HYQ_D + c0;
    double s = 0.0;
    for (int r0 = 0; r0 < t; r0 += MEAN_ROWS) {
        const int rows = min(MEAN_ROWS, t - r0);
        __syncthreads();
        // 16 threads per row, 4 bytes each
        for (int e = threadIdx.x; e < rows * (MEAN_CH / 2); e += MEAN_THREADS) {
            const int r = e / (MEAN_CH / 2), c2 = (e % (MEAN_CH / 2)) * 2;
            *reinterpret_cast<uint32_t*>(&tile[r][c2]) = __ldg(reinterpret_cast<const uint32_t*>(base + (long)(r0 + r) * HYQ_D + c2));
        }
        __syncthreads();
        if (threadIdx.x < MEAN_CH) {
            int r = 0;
            for (; r + 8 <= rows; r += 8) {
                float v[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) v[j] = __bfloat162float(tile[r + j][threadIdx.x]);
#pragma unroll
                for (int j = 0; j < 8; ++j) s += (double)v[j];
            }
            for (; r < rows; ++r) s += (double)__bfloat162float(tile[r][threadIdx.x]);
        }
    }
    if (threadIdx.x < MEAN_CH) qbar[bh * HYQ_D + c0 + threadIdx.x] = s / (double)t;
}

// -------------------------------------------------------------------------------------------
constexpr int KROW_WORDS = HYQ_D / 2 + 1;    // 65 words per staged key row: conflict-free column reads

__global__ void __launch_bounds__(SCORE_KEYS)
vscore_kernel(const __nv_bfloat16* __restrict__ kmat, const double* __restrict__ qbar, int Hq, int Hkv, int Lk,
              int P, double* __restrict__ scores) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int g = Hq / Hkv;
    uint32_t* ktile = reinterpret_cast<uint32_t*>(smem_raw);                          // [SCORE_KEYS][KROW_WORDS]
    double* qs = reinterpret_cast<double*>(smem_raw + align_up(SCORE_KEYS * KROW_WORDS * 4, 16));  // [g][D]

    const int p0 = blockIdx.x * SCORE_KEYS;
    const int kvh = blockIdx.y, b = blockIdx.z;
    const int n_keys = min(SCORE_KEYS, P - p0);

    // stage the K rows (coalesced 16-byte reads, 4-byte shared stores)
    const uint4* src = reinterpret_cast<const uint4*>(kmat + (((long)b * Hkv + kvh) * Lk + p0) * HYQ_D);
    for (int v = threadIdx.x; v < n_keys * (HYQ_D / 8); v += SCORE_KEYS) {
        const uint4 w = __ldg(src + v);
        const int row = v / (HYQ_D / 8), c4 = (v % (HYQ_D / 8)) * 4;
        uint32_t* dst = ktile + row * KROW_WORDS + c4;
        dst[0] = w.x; dst[1] = w.y; dst[2] = w.z; dst[3] = w.w;
    }
    for (int e = threadIdx.x; e < g * HYQ_D; e += SCORE_KEYS)
        qs[e] = qbar[((long)b * Hq + (long)kvh * g) * HYQ_D + e];
    __syncthreads();
    if ((int)threadIdx.x >= n_keys) return;

    const uint32_t* krow = ktile + threadIdx.x * KROW_WORDS;
    for (int r0 = 0; r0 < g; r0 += SCORE_GC) {
        double s[SCORE_GC];
        const double* qr[SCORE_GC];
#pragma unroll
        for (int c = 0; c < SCORE_GC; ++c) { s[c] = 0.0; qr[c] = qs + min(r0 + c, g - 1) * HYQ_D; }
#pragma unroll 4
        for (int w = 0; w < HYQ_D / 2; ++w) {
            const uint32_t kw = krow[w];
            const double k0 = (double)bf16_lo(kw), k1 = (double)bf16_hi(kw);
#pragma unroll
            for (int c = 0; c < SCORE_GC; ++c) {
                s[c] = fma(qr[c][2 * w], k0, s[c]);
                s[c] = fma(qr[c][2 * w + 1], k1, s[c]);
            }
        }
#pragma unroll
        for (int c = 0; c < SCORE_GC; ++c)
            if (r0 + c < g) scores[(((long)b * Hq + (long)kvh * g + r0 + c)) * P + p0 + threadIdx.x] = s[c];
    }
}

// -------------------------------------------------------------------------------------------
// larger score <=> larger key; -0 and +0 map to the same key
__device__ __forceinline__ unsigned long long order_key(double s) {
    unsigned long long u = (s == 0.0) ? 0ull : (unsigned long long)__double_as_longlong(s);
    return (u >> 63) ? ~u : (u | 0x8000000000000000ull);
}

// One CTA per (b, query head); every warp owns a contiguous segment of the row (coalesced reads, no CTA-wide
// synchronisation inside a scan of the row).
__global__ void __launch_bounds__(TOPK_THREADS)
topk_kernel(const double* __restrict__ scores, int P, int k, int32_t* __restrict__ idx_out) {
    constexpr int NW = TOPK_THREADS / 32;
    __shared__ int whist[NW][256];                     // one digit histogram per warp (no contention across warps)
    __shared__ int hist[256];
    __shared__ int warp_gt[NW], warp_eq[NW];
    __shared__ unsigned long long sh_prefix;
    __shared__ int sh_krem, sh_bin, n_cand;
    __shared__ unsigned long long cand[TOPK_CAND];     // the keys still in the race once few are left
    const double* row = scores + (long)blockIdx.x * P;
    int32_t* out = idx_out + (long)blockIdx.x * k;
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const int per = (P + NW - 1) / NW;
    const int seg0 = min(P, wid * per), seg1 = min(P, seg0 + per);

    // radix select: after the loop `prefix` is the key of the k-th largest score and k_rem how
    // many positions holding exactly that key are still to be taken
    // Once a pass leaves no more than TOPK_CAND keys sharing the digits fixed so far, those keys are gathered into
    // shared memory (one more sweep over the row) and the remaining passes run over that short list.
    unsigned long long prefix = 0ull;
    int k_rem = k;
    bool gathered = false;
    for (int pass = 0; pass < 8; ++pass) {
        const int shift = 56 - 8 * pass;
#pragma unroll
        for (int e = 0; e < 8; ++e) whist[wid][lane + 32 * e] = 0;
        __syncwarp();
        if (gathered) {
            const int nc = n_cand;
            for (int c = threadIdx.x; c < nc; c += TOPK_THREADS) {
                const unsigned long long key = cand[c];
                if ((key >> (shift + 8)) == (prefix >> (shift + 8))) atomicAdd(&whist[wid][(int)((key >> shift) & 0xFF)], 1);
            }
        } else {
            // (eight loads in flight per thread: a scan of the row is bound by their latency)
            for (int p0 = seg0 + lane; p0 < seg1; p0 += 32 * SCAN_DEPTH) {
                double v[SCAN_DEPTH];
#pragma unroll
                for (int j = 0; j < SCAN_DEPTH; ++j) v[j] = (p0 + 32 * j < seg1) ? __ldg(row + p0 + 32 * j) : 0.0;
#pragma unroll
                for (int j = 0; j < SCAN_DEPTH; ++j) {
                    const unsigned long long key = order_key(v[j]);
                    if (p0 + 32 * j < seg1 && (pass == 0 || (key >> (shift + 8)) == (prefix >> (shift + 8))))
                        atomicAdd(&whist[wid][(int)((key >> shift) & 0xFF)], 1);
                }
            }
        }
        __syncthreads();
        if (threadIdx.x < 256) {
            int tot = 0;
#pragma unroll 8
            for (int w = 0; w < NW; ++w) tot += whist[w][threadIdx.x];
            hist[threadIdx.x] = tot;
        }
        __syncthreads();
        // the digit d whose bin holds the k_rem-th largest candidate: the largest d with
        // count(bins above d) < k_rem <= count(bins d and above); lane l of warp 0 looks at bins 255-8l .. 248-8l
        if (wid == 0) {
            const int hi = 255 - 8 * lane;
            int mine = 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) mine += hist[hi - j];
            int incl = mine;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int v = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += v;
            }
            int above = incl - mine;                   // candidates in bins above this lane's eight
            if (above < k_rem && k_rem <= incl) {      // exactly one lane (the candidates number at least k_rem)
                int d = hi;
                for (; d > hi - 7; --d) {
                    if (above + hist[d] >= k_rem) break;
                    above += hist[d];
                }
                sh_prefix = prefix | ((unsigned long long)d << shift);
                sh_krem = k_rem - above;
                sh_bin = hist[d];                      // keys that share all digits fixed so far
                if (!gathered) n_cand = 0;
            }
        }
        __syncthreads();
        prefix = sh_prefix;
        k_rem = sh_krem;
        if (!gathered && pass < 6 && sh_bin <= TOPK_CAND) {
            for (int p0 = seg0 + lane; p0 < seg1; p0 += 32 * SCAN_DEPTH) {
                double v[SCAN_DEPTH];
#pragma unroll
                for (int j = 0; j < SCAN_DEPTH; ++j) v[j] = (p0 + 32 * j < seg1) ? __ldg(row + p0 + 32 * j) : 0.0;
#pragma unroll
                for (int j = 0; j < SCAN_DEPTH; ++j) {
                    const unsigned long long key = order_key(v[j]);
                    if (p0 + 32 * j < seg1 && (key >> shift) == (prefix >> shift)) cand[atomicAdd(&n_cand, 1)] = key;
                }
            }
            gathered = true;                           // (uniform over the CTA: sh_bin is)
            __syncthreads();
        }
    }

    // ordered compaction: positions ascending; among keys equal to the threshold the first k_rem.
    // Scan 1 counts, per warp segment, the keys above and equal to the threshold; scan 2 writes: the output
    // slot of a selected position = (keys above the threshold before it) + min(keys equal before it, k_rem).
    int n_gt = 0, n_eq = 0;
    for (int base = seg0; base < seg1; base += 32 * SCAN_DEPTH) {
        double v[SCAN_DEPTH];
#pragma unroll
        for (int j = 0; j < SCAN_DEPTH; ++j) v[j] = (base + 32 * j + lane < seg1) ? __ldg(row + base + 32 * j + lane) : 0.0;
#pragma unroll
        for (int j = 0; j < SCAN_DEPTH; ++j) {
            const bool live = base + 32 * j + lane < seg1;
            const unsigned long long key = order_key(v[j]);
            n_gt += __popc(__ballot_sync(0xffffffffu, live && key > prefix));
            n_eq += __popc(__ballot_sync(0xffffffffu, live && key == prefix));
        }
    }
    if (lane == 0) { warp_gt[wid] = n_gt; warp_eq[wid] = n_eq; }
    __syncthreads();
    int gt_run = 0, eq_run = 0;
    for (int w = 0; w < wid; ++w) { gt_run += warp_gt[w]; eq_run += warp_eq[w]; }
    const unsigned lt_mask = (1u << lane) - 1u;
    for (int base = seg0; base < seg1; base += 32 * SCAN_DEPTH) {
        double v[SCAN_DEPTH];
#pragma unroll
        for (int j = 0; j < SCAN_DEPTH; ++j) v[j] = (base + 32 * j + lane < seg1) ? __ldg(row + base + 32 * j + lane) : 0.0;
#pragma unroll
        for (int j = 0; j < SCAN_DEPTH; ++j) {
            const int p = base + 32 * j + lane;
            const bool live = p < seg1;
            const unsigned long long key = order_key(v[j]);
            const bool gt = live && key > prefix, eq = live && key == prefix;
            const unsigned b_gt = __ballot_sync(0xffffffffu, gt), b_eq = __ballot_sync(0xffffffffu, eq);
            const int eq_rank = eq_run + __popc(b_eq & lt_mask);
            const int pos = gt_run + __popc(b_gt & lt_mask) + min(eq_rank, k_rem);
            if ((gt || (eq && eq_rank < k_rem)) && pos < k) out[pos] = p;
            gt_run += __popc(b_gt);
            eq_run += __popc(b_eq);
        }
    }
}

// -------------------------------------------------------------------------------------------
size_t select_workspace_bytes(int B, int Hq, int Lk, int window) {
    const long P = (Lk - window > 0) ? Lk - window : 0;
    return align_up((size_t)B * Hq * HYQ_D * sizeof(double), 256) + align_up((size_t)B * Hq * P * sizeof(double), 256);
}

int launch_select(const void* q, const void* k, int B, int Hq, int Hkv, int Lq, int Lk, int window, int n_tail,
                  int k_sel, int32_t* idx_out, void* ws, cudaStream_t st) {
    const int P = (Lk - window > 0) ? Lk - window : 0;
    const int t = n_tail ? n_tail : (window < Lq ? window : Lq);
    const int g = Hq / Hkv;
    double* qbar = static_cast<double*>(ws);
    double* scores = reinterpret_cast<double*>(static_cast<char*>(ws) + align_up((size_t)B * Hq * HYQ_D * sizeof(double), 256));

    tail_mean_kernel<<<dim3(B * Hq, HYQ_D / MEAN_CH), MEAN_THREADS, 0, st>>>(static_cast<const __nv_bfloat16*>(q), Lq, t, qbar);
    if (launch_status() != HYQ_OK) return HYQ_ERR_CUDA;

    const size_t smem = align_up(SCORE_KEYS * KROW_WORDS * 4, 16) + (size_t)g * HYQ_D * sizeof(double);
    if (smem > 200 * 1024) return HYQ_ERR_UNSUPPORTED;
    if (smem > 48 * 1024 &&
        cudaFuncSetAttribute(vscore_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return HYQ_ERR_CUDA;
    const dim3 grid((P + SCORE_KEYS - 1) / SCORE_KEYS, Hkv, B);
    vscore_kernel<<<grid, SCORE_KEYS, smem, st>>>(static_cast<const __nv_bfloat16*>(k), qbar, Hq, Hkv, Lk, P, scores);
    if (launch_status() != HYQ_OK) return HYQ_ERR_CUDA;

    topk_kernel<<<B * Hq, TOPK_THREADS, 0, st>>>(scores, P, k_sel, idx_out);
    return launch_status();
}

// top-k of `rows` score rows of length P (shared with the column-mass selector)
int launch_topk(const double* scores, long rows, int P, int k_sel, int32_t* idx_out, cudaStream_t st) {
    topk_kernel<<<(unsigned)rows, TOPK_THREADS, 0, st>>>(scores, P, k_sel, idx_out);
    return launch_status();
}

// -------------------------------------------------------------------------------------------
// Selection without caller-provided scratch: the tail means and the fp64 scores live in a fixed array
// that is part of the library image on every device that loads it.
static __device__ __align__(256) unsigned char g_select_scratch[HYQ_SELECT_STATIC_SCRATCH_BYTES];

// Device address of g_select_scratch on the current device.  In host code the array's name is only
// a handle for the runtime, never a pointer a kernel may use, so the address is looked up once per
// device (with that device current) and cached.
static int select_static_scratch(void** out) {
    constexpr int MAX_DEVICES = 64;
    static std::mutex mu;
    static void* cached[MAX_DEVICES] = {};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return HYQ_ERR_CUDA;
    std::lock_guard<std::mutex> lock(mu);
    if (cached[dev] == nullptr) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_select_scratch) != cudaSuccess || ptr == nullptr) return HYQ_ERR_CUDA;
        cached[dev] = ptr;
    }
    *out = cached[dev];
    return HYQ_OK;
}

int launch_select_static(const void* q, const void* k, int B, int Hq, int Hkv, int Lq, int Lk, int window, int n_tail,
                         int k_sel, int32_t* idx_out, cudaStream_t st) {
    if (select_workspace_bytes(B, Hq, Lk, window) > (size_t)HYQ_SELECT_STATIC_SCRATCH_BYTES) return HYQ_ERR_WORKSPACE;
    void* scratch = nullptr;
    const int rc = select_static_scratch(&scratch);
    if (rc != HYQ_OK) return rc;
    // every byte of scratch that the kernels read is written earlier in the same call, so nothing has to
    // be cleared between calls
    return launch_select(q, k, B, Hq, Hkv, Lq, Lk, window, n_tail, k_sel, idx_out, scratch, st);
}

}  // namespace hyq
