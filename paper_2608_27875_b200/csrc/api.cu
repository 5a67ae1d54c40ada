// C-ABI entry points of the hyq library: argument checks on the host, then kernel launches.
#include <cmath>

#include "attn_common.cuh"

namespace hyq {
size_t attn_simt_workspace_bytes(const hyq_attn_args& a);
int launch_attn_simt(const hyq_attn_args& a, float alpha, cudaStream_t st);
size_t attn_tc_workspace_bytes(const hyq_attn_args& a);
int launch_attn_tc(const hyq_attn_args& a, float alpha, cudaStream_t st);
int tc_restarts(unsigned long long* count, bool reset);
namespace tcbt {
int launch_attn_tc(const hyq_attn_args& a, float alpha, cudaStream_t st);     // 32- and 128-token quantization blocks
int tc_restarts(unsigned long long* count, bool reset);
}
}  // namespace hyq

namespace hyq {
static TcTestHooks g_tc_hooks = {0, -1};
TcTestHooks tc_test_hooks() { return g_tc_hooks; }
}  // namespace hyq

using namespace hyq;

extern "C" {

const char* hyq_status_string(int status) {
    switch (status) {
        case HYQ_OK: return "ok";
        case HYQ_ERR_INVALID_ARG: return "invalid argument";
        case HYQ_ERR_UNSUPPORTED: return "unsupported shape or format";
        case HYQ_ERR_WORKSPACE: return "workspace too small";
        case HYQ_ERR_ALIGNMENT: return "pointer not 16-byte aligned";
        case HYQ_ERR_CUDA: return "CUDA call failed";
        case HYQ_ERR_TIMEOUT: return "bounded device wait expired";
        default: return "unknown status";
    }
}

int hyq_version(void) { return 2; }   // 2: decode side, column-mass selector, block sizes

int hyq_test_set_attention_hooks(long long wait_limit_clocks, int drop_load_position) {
    if (wait_limit_clocks < 0 || drop_load_position < -1) return HYQ_ERR_INVALID_ARG;
    g_tc_hooks.wait_limit = wait_limit_clocks;
    g_tc_hooks.drop_load = drop_load_position;
    return HYQ_OK;
}

int hyq_test_read_attention_restarts(unsigned long long* count_out, int reset) {
    if (!count_out) return HYQ_ERR_INVALID_ARG;
    unsigned long long a = 0ull, b = 0ull;
    if (tc_restarts(&a, reset != 0) != HYQ_OK || tcbt::tc_restarts(&b, reset != 0) != HYQ_OK) return HYQ_ERR_CUDA;
    *count_out = a + b;
    return HYQ_OK;
}

int hyq_paper_k(int Lk, int window, double ratio) {
    const long P = (Lk - window > 0) ? (long)Lk - window : 0;
    if (P == 0) return 0;
    long k = (long)std::ceil((double)P * ratio);
    if (k < 1) k = 1;
    if (k > P) k = P;
    return (int)k;
}

static int check_select(const void* q, const void* k_, int B, int Hq, int Hkv, int Lq, int Lk, int D, int window,
                        int n_tail, int k) {
    if (B <= 0 || Hq <= 0 || Hkv <= 0 || Lq <= 0 || Lk <= 0 || window < 0 || k < 0 || n_tail < 0) return HYQ_ERR_INVALID_ARG;
    if (Hq % Hkv) return HYQ_ERR_INVALID_ARG;
    if (D != HYQ_D) return HYQ_ERR_UNSUPPORTED;
    const long P = (Lk - window > 0) ? (long)Lk - window : 0;
    if (P == 0 || k == 0) return HYQ_OK;
    if (k > P || n_tail > Lq) return HYQ_ERR_INVALID_ARG;
    if (n_tail == 0 && window == 0) return HYQ_ERR_INVALID_ARG;    // mean of zero rows
    (void)q; (void)k_;
    return HYQ_OK;
}

int hyq_select_vertical_workspace(int B, int Hq, int Hkv, int Lq, int Lk, int D, int window, int k, size_t* bytes) {
    if (!bytes) return HYQ_ERR_INVALID_ARG;
    const int rc = check_select(nullptr, nullptr, B, Hq, Hkv, Lq, Lk, D, window, 1, k);
    if (rc != HYQ_OK) return rc;
    *bytes = select_workspace_bytes(B, Hq, Lk, window);
    return HYQ_OK;
}

int hyq_select_vertical(const void* q, const void* k_, int B, int Hq, int Hkv, int Lq, int Lk, int D, int window,
                        int n_tail, int k, int32_t* idx_out, void* workspace, size_t workspace_bytes, void* stream) {
    const int rc = check_select(q, k_, B, Hq, Hkv, Lq, Lk, D, window, n_tail, k);
    if (rc != HYQ_OK) return rc;
    const long P = (Lk - window > 0) ? (long)Lk - window : 0;
    if (P == 0 || k == 0) return HYQ_OK;
    if (!q || !k_ || !idx_out || !workspace) return HYQ_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k_) || !aligned16(workspace) || (reinterpret_cast<uintptr_t>(idx_out) & 3u))
        return HYQ_ERR_ALIGNMENT;
    if (workspace_bytes < select_workspace_bytes(B, Hq, Lk, window)) return HYQ_ERR_WORKSPACE;
    return launch_select(q, k_, B, Hq, Hkv, Lq, Lk, window, n_tail, k, idx_out, workspace, static_cast<cudaStream_t>(stream));
}

int hyq_select_vertical_static(const void* q, const void* k_, int B, int Hq, int Hkv, int Lq, int Lk, int D, int window,
                               int n_tail, int k, int32_t* idx_out, void* stream) {
    const int rc = check_select(q, k_, B, Hq, Hkv, Lq, Lk, D, window, n_tail, k);
    if (rc != HYQ_OK) return rc;
    const long P = (Lk - window > 0) ? (long)Lk - window : 0;
    if (P == 0 || k == 0) return HYQ_OK;
    if (!q || !k_ || !idx_out) return HYQ_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k_) || (reinterpret_cast<uintptr_t>(idx_out) & 3u)) return HYQ_ERR_ALIGNMENT;
    return launch_select_static(q, k_, B, Hq, Hkv, Lq, Lk, window, n_tail, k, idx_out, static_cast<cudaStream_t>(stream));
}

static int check_select_mass(int B, int Hq, int Hkv, int Lq, int Lk, int D, int window, int n_queries, int k, int* n_eff) {
    if (n_queries < 0) return HYQ_ERR_INVALID_ARG;
    const int rc = check_select(nullptr, nullptr, B, Hq, Hkv, Lq, Lk, D, window, n_queries, k);
    if (rc != HYQ_OK) return rc;
    const int tail = window < Lq ? window : Lq;
    *n_eff = n_queries ? n_queries : tail;
    const long P = (Lk - window > 0) ? (long)Lk - window : 0;
    if (P == 0 || k == 0) return HYQ_OK;
    if (Lq > Lk || *n_eff > tail || *n_eff <= 0) return HYQ_ERR_INVALID_ARG;
    return HYQ_OK;
}

int hyq_select_vertical_mass_workspace(int B, int Hq, int Hkv, int Lq, int Lk, int D, int window, int n_queries, int k,
                                       size_t* bytes) {
    if (!bytes) return HYQ_ERR_INVALID_ARG;
    int nT = 0;
    const int rc = check_select_mass(B, Hq, Hkv, Lq, Lk, D, window, n_queries, k, &nT);
    if (rc != HYQ_OK) return rc;
    *bytes = select_mass_workspace_bytes(B, Hq, Lk, window, nT);
    return HYQ_OK;
}

int hyq_select_vertical_mass(const void* q, const void* k_, int B, int Hq, int Hkv, int Lq, int Lk, int D, int window,
                             int n_queries, int k, float softmax_scale, int32_t* idx_out, void* workspace,
                             size_t workspace_bytes, void* stream) {
    int nT = 0;
    const int rc = check_select_mass(B, Hq, Hkv, Lq, Lk, D, window, n_queries, k, &nT);
    if (rc != HYQ_OK) return rc;
    const long P = (Lk - window > 0) ? (long)Lk - window : 0;
    if (P == 0 || k == 0) return HYQ_OK;
    if (!q || !k_ || !idx_out || !workspace) return HYQ_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k_) || !aligned16(workspace) || (reinterpret_cast<uintptr_t>(idx_out) & 3u))
        return HYQ_ERR_ALIGNMENT;
    if (workspace_bytes < select_mass_workspace_bytes(B, Hq, Lk, window, nT)) return HYQ_ERR_WORKSPACE;
    const double alpha = softmax_scale != 0.0f ? (double)softmax_scale : 1.0 / std::sqrt((double)D);
    return launch_select_mass(q, k_, B, Hq, Hkv, Lq, Lk, window, nT, k, alpha, idx_out, workspace,
                              static_cast<cudaStream_t>(stream));
}

int hyq_quantize_blocks(const void* x, int B, int H, int L, int D, int block_tokens, int format, void* codes_out,
                        float* scales_out, void* stream) {
    if (B <= 0 || H <= 0 || L <= 0) return HYQ_ERR_INVALID_ARG;
    if (!x || !codes_out || !scales_out) return HYQ_ERR_INVALID_ARG;
    if (D != HYQ_D || !block_tokens_ok(block_tokens)) return HYQ_ERR_UNSUPPORTED;
    if (format != HYQ_FMT_INT8 && format != HYQ_FMT_FP8_E4M3 && format != HYQ_FMT_INT4) return HYQ_ERR_UNSUPPORTED;
    if (!aligned16(x) || !aligned16(codes_out) || (reinterpret_cast<uintptr_t>(scales_out) & 3u)) return HYQ_ERR_ALIGNMENT;
    return launch_quantize(x, (long)B * H, L, block_tokens, format, codes_out, scales_out, static_cast<cudaStream_t>(stream));
}

static int check_attn(const hyq_attn_args* a, bool need_pointers) {
    if (!a || a->struct_size != sizeof(hyq_attn_args)) return HYQ_ERR_INVALID_ARG;
    if (a->B <= 0 || a->Hq <= 0 || a->Hkv <= 0 || a->L <= 0 || a->window < 0 || a->k < 0) return HYQ_ERR_INVALID_ARG;
    if (a->Hq % a->Hkv || a->k > a->L || a->Lq < 0 || a->Lq > a->L) return HYQ_ERR_INVALID_ARG;
    if (a->window_mode != HYQ_WINDOW_SLIDING && a->window_mode != HYQ_WINDOW_FIXED_TAIL) return HYQ_ERR_INVALID_ARG;
    if (a->out_dtype != 0 && a->out_dtype != 1) return HYQ_ERR_INVALID_ARG;
    if (a->impl < HYQ_IMPL_AUTO || a->impl > HYQ_IMPL_SIMT) return HYQ_ERR_INVALID_ARG;
    if (a->D != HYQ_D || !block_tokens_ok(a->block_tokens)) return HYQ_ERR_UNSUPPORTED;
    const bool int8 = a->q_format == HYQ_FMT_INT8 && a->k_format == HYQ_FMT_INT8 && a->v_format == HYQ_FMT_INT8;
    const bool int4 = a->q_format == HYQ_FMT_INT4 && a->k_format == HYQ_FMT_INT4 && a->v_format == HYQ_FMT_FP8_E4M3;
    const bool fp8 = a->q_format == HYQ_FMT_FP8_E4M3 && a->k_format == HYQ_FMT_FP8_E4M3 && a->v_format == HYQ_FMT_FP8_E4M3;
    if (!int8 && !int4 && !fp8) return HYQ_ERR_UNSUPPORTED;
    if (!need_pointers) return HYQ_OK;
    const void* ptrs[] = {a->q, a->k_, a->v, a->q_codes, a->k_codes, a->v_codes, a->q_scales, a->k_scales, a->v_scales, a->out};
    for (const void* p : ptrs)
        if (!p) return HYQ_ERR_INVALID_ARG;
    if (a->k > 0 && !a->vl_idx) return HYQ_ERR_INVALID_ARG;
    const void* al[] = {a->q, a->k_, a->v, a->q_codes, a->k_codes, a->v_codes, a->out, a->workspace};
    for (const void* p : al)
        if (!aligned16(p)) return HYQ_ERR_ALIGNMENT;
    return HYQ_OK;
}

static bool use_simt(const hyq_attn_args* a) { return a->impl == HYQ_IMPL_SIMT; }

int hyq_hybrid_attention_prefill_workspace(const hyq_attn_args* args, size_t* bytes) {
    if (!bytes) return HYQ_ERR_INVALID_ARG;
    const int rc = check_attn(args, false);
    if (rc != HYQ_OK) return rc;
    *bytes = use_simt(args) ? attn_simt_workspace_bytes(*args) : attn_tc_workspace_bytes(*args);
    return HYQ_OK;
}

int hyq_hybrid_attention_prefill(const hyq_attn_args* args, void* stream) {
    const int rc = check_attn(args, true);
    if (rc != HYQ_OK) return rc;
    const size_t need = use_simt(args) ? attn_simt_workspace_bytes(*args) : attn_tc_workspace_bytes(*args);
    if (need > 0 && (!args->workspace || args->workspace_bytes < need)) return HYQ_ERR_WORKSPACE;
    const float alpha = args->softmax_scale != 0.0f ? args->softmax_scale : 1.0f / sqrtf((float)args->D);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (use_simt(args)) return launch_attn_simt(*args, alpha, st);
    return args->block_tokens == HYQ_BLOCK_TOKENS ? launch_attn_tc(*args, alpha, st) : tcbt::launch_attn_tc(*args, alpha, st);
}

// ---- ragged batches: the plain calls, sequence by sequence, on packed buffers ---------------------------------
static int check_cu(int n_seq, const int32_t* cu) {
    if (n_seq <= 0 || !cu || cu[0] != 0) return HYQ_ERR_INVALID_ARG;
    for (int s = 0; s < n_seq; ++s)
        if (cu[s + 1] <= cu[s]) return HYQ_ERR_INVALID_ARG;
    return HYQ_OK;
}

// sequence numbers, longest first (ties by position)
static void longest_first(int n_seq, const int32_t* cu, int* order) {
    for (int s = 0; s < n_seq; ++s) order[s] = s;
    for (int a = 1; a < n_seq; ++a) {                       // insertion sort: batches are small
        const int v = order[a], lv = cu[v + 1] - cu[v];
        int b = a - 1;
        while (b >= 0 && cu[order[b] + 1] - cu[order[b]] < lv) { order[b + 1] = order[b]; --b; }
        order[b + 1] = v;
    }
}

int hyq_select_vertical_varlen(const void* q, const void* k_, int n_seq, const int32_t* cu, int Hq, int Hkv, int D,
                               int window, int n_tail, const int32_t* k_per_seq, int32_t* idx_out, void* workspace,
                               size_t workspace_bytes, void* stream) {
    int rc = check_cu(n_seq, cu);
    if (rc != HYQ_OK) return rc;
    if (!k_per_seq) return HYQ_ERR_INVALID_ARG;
    size_t need = 0;
    for (int s = 0; s < n_seq; ++s) {
        const int L = cu[s + 1] - cu[s];
        rc = check_select(q, k_, 1, Hq, Hkv, L, L, D, window, n_tail, k_per_seq[s]);
        if (rc != HYQ_OK) return rc;
        const long P = L - window > 0 ? (long)L - window : 0;
        if (P > 0 && k_per_seq[s] > 0) need = need > select_workspace_bytes(1, Hq, L, window) ? need : select_workspace_bytes(1, Hq, L, window);
    }
    if (need == 0) return HYQ_OK;
    if (!q || !k_ || !idx_out || !workspace) return HYQ_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k_) || !aligned16(workspace) || (reinterpret_cast<uintptr_t>(idx_out) & 3u)) return HYQ_ERR_ALIGNMENT;
    if (workspace_bytes < need) return HYQ_ERR_WORKSPACE;
    int* order = new int[n_seq];
    long* koff = new long[n_seq];
    long acc = 0;
    for (int s = 0; s < n_seq; ++s) { koff[s] = acc; acc += k_per_seq[s]; }
    longest_first(n_seq, cu, order);
    for (int n = 0; n < n_seq && rc == HYQ_OK; ++n) {
        const int s = order[n], L = cu[s + 1] - cu[s], ks = k_per_seq[s];
        if (ks == 0 || L - window <= 0) continue;
        const char* qs = static_cast<const char*>(q) + (size_t)Hq * D * cu[s] * 2;
        const char* kk = static_cast<const char*>(k_) + (size_t)Hkv * D * cu[s] * 2;
        rc = launch_select(qs, kk, 1, Hq, Hkv, L, L, window, n_tail, ks, idx_out + (size_t)Hq * koff[s], workspace,
                           static_cast<cudaStream_t>(stream));
    }
    delete[] order;
    delete[] koff;
    return rc;
}

int hyq_quantize_blocks_varlen(const void* x, int n_seq, const int32_t* cu, int H, int D, int block_tokens, int format,
                               void* codes_out, float* scales_out, void* stream) {
    int rc = check_cu(n_seq, cu);
    if (rc != HYQ_OK) return rc;
    if (H <= 0 || !x || !codes_out || !scales_out) return HYQ_ERR_INVALID_ARG;
    if (D != HYQ_D || !block_tokens_ok(block_tokens)) return HYQ_ERR_UNSUPPORTED;
    if (format != HYQ_FMT_INT8 && format != HYQ_FMT_FP8_E4M3 && format != HYQ_FMT_INT4) return HYQ_ERR_UNSUPPORTED;
    if (!aligned16(x) || !aligned16(codes_out) || (reinterpret_cast<uintptr_t>(scales_out) & 3u)) return HYQ_ERR_ALIGNMENT;
    const size_t row_bytes = format == HYQ_FMT_INT4 ? D / 2 : D;
    size_t nb_before = 0;
    for (int s = 0; s < n_seq && rc == HYQ_OK; ++s) {
        const int L = cu[s + 1] - cu[s];
        rc = launch_quantize(static_cast<const char*>(x) + (size_t)H * D * cu[s] * 2, H, L, block_tokens, format,
                             static_cast<char*>(codes_out) + (size_t)H * row_bytes * cu[s], scales_out + (size_t)H * nb_before,
                             static_cast<cudaStream_t>(stream));
        nb_before += (size_t)(L + block_tokens - 1) / block_tokens;
    }
    return rc;
}

int hyq_hybrid_attention_prefill_varlen(const hyq_attn_args* args, int n_seq, const int32_t* cu, const int32_t* k_per_seq,
                                        void* stream) {
    int rc = check_cu(n_seq, cu);
    if (rc != HYQ_OK) return rc;
    if (!args || args->struct_size != sizeof(hyq_attn_args) || !k_per_seq) return HYQ_ERR_INVALID_ARG;
    const int bt = args->block_tokens;
    if (!block_tokens_ok(bt)) return HYQ_ERR_UNSUPPORTED;
    const size_t q_row = args->q_format == HYQ_FMT_INT4 ? HYQ_D / 2 : HYQ_D, k_row = args->k_format == HYQ_FMT_INT4 ? HYQ_D / 2 : HYQ_D;
    const size_t v_row = args->v_format == HYQ_FMT_INT4 ? HYQ_D / 2 : HYQ_D;
    // one argument block per sequence, all checked before the first launch
    hyq_attn_args* per = new hyq_attn_args[n_seq];
    int* order = new int[n_seq];
    size_t nb_before = 0, k_before = 0;
    for (int s = 0; s < n_seq && rc == HYQ_OK; ++s) {
        const int L = cu[s + 1] - cu[s];
        hyq_attn_args a = *args;
        a.B = 1; a.L = L; a.Lq = 0; a.k = k_per_seq[s];
        const size_t t0 = (size_t)cu[s];
        auto at = [](const void* base, size_t bytes) -> const void* { return base ? static_cast<const char*>(base) + bytes : nullptr; };
        a.q = at(args->q, (size_t)args->Hq * HYQ_D * t0 * 2);
        a.k_ = at(args->k_, (size_t)args->Hkv * HYQ_D * t0 * 2);
        a.v = at(args->v, (size_t)args->Hkv * HYQ_D * t0 * 2);
        a.q_codes = at(args->q_codes, (size_t)args->Hq * q_row * t0);
        a.k_codes = at(args->k_codes, (size_t)args->Hkv * k_row * t0);
        a.v_codes = at(args->v_codes, (size_t)args->Hkv * v_row * t0);
        a.q_scales = args->q_scales ? args->q_scales + (size_t)args->Hq * nb_before : nullptr;
        a.k_scales = args->k_scales ? args->k_scales + (size_t)args->Hkv * nb_before : nullptr;
        a.v_scales = args->v_scales ? args->v_scales + (size_t)args->Hkv * nb_before : nullptr;
        a.vl_idx = (args->vl_idx && a.k > 0) ? args->vl_idx + (size_t)args->Hq * k_before : nullptr;
        a.out = const_cast<void*>(at(args->out, (size_t)args->Hq * HYQ_D * t0 * (args->out_dtype == 1 ? 4 : 2)));
        a.lse = args->lse ? args->lse + (size_t)args->Hq * t0 : nullptr;
        if (a.k < 0 || a.k > (L - a.window > 0 ? L - a.window : 0)) rc = HYQ_ERR_INVALID_ARG;
        if (rc == HYQ_OK) rc = check_attn(&a, true);
        if (rc == HYQ_OK) {
            const size_t need = use_simt(&a) ? attn_simt_workspace_bytes(a) : attn_tc_workspace_bytes(a);
            if (need > 0 && (!a.workspace || a.workspace_bytes < need)) rc = HYQ_ERR_WORKSPACE;
        }
        per[s] = a;
        nb_before += (size_t)(L + bt - 1) / bt;
        k_before += (size_t)k_per_seq[s];
    }
    if (rc == HYQ_OK) {
        longest_first(n_seq, cu, order);
        for (int n = 0; n < n_seq && rc == HYQ_OK; ++n) rc = hyq_hybrid_attention_prefill(&per[order[n]], stream);
    }
    delete[] per;
    delete[] order;
    return rc;
}

}  // extern "C"
