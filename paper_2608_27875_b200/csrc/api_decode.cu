// C-ABI entry points of the decode side: argument checks on the host, then kernel launches.
#include <cmath>

#include "decode_common.cuh"

using namespace hyq;

static int check_cache(const hyq_kv_cache* c, bool need_pointers) {
    if (!c || c->struct_size != sizeof(hyq_kv_cache)) return HYQ_ERR_INVALID_ARG;
    if (c->B <= 0 || c->Hq <= 0 || c->Hkv <= 0 || c->N <= 0 || c->window < 0 || c->k < 0) return HYQ_ERR_INVALID_ARG;
    if (c->Hq % c->Hkv) return HYQ_ERR_INVALID_ARG;
    if (c->staging_capacity < 0 || c->n_staging < 0 || c->n_staging > c->staging_capacity) return HYQ_ERR_INVALID_ARG;
    if (c->D != HYQ_D || (c->group != 32 && c->group != 64 && c->group != 128) ||
        (c->format != HYQ_FMT_INT4 && c->format != HYQ_FMT_INT8 && c->format != HYQ_FMT_FP8_E4M3) ||
        c->Hq / c->Hkv > 8 * DEC_MAX_GROUP)
        return HYQ_ERR_UNSUPPORTED;
    const CacheGeo g = cache_geo(*c);
    if (c->k > c->N - g.W) return HYQ_ERR_INVALID_ARG;
    if ((long)c->B * c->Hkv * ((c->Hq / c->Hkv + DEC_MAX_GROUP - 1) / DEC_MAX_GROUP) > 65535) return HYQ_ERR_UNSUPPORTED;
    if (c->cap_quantized_rows < 0 || c->cap_vertical < 0 || c->cap_window < 0) return HYQ_ERR_INVALID_ARG;
    if ((c->cap_quantized_rows && (c->cap_quantized_rows % c->group || c->cap_quantized_rows < g.nQp)) ||
        (c->cap_vertical && c->cap_vertical < c->k) || (c->cap_window && c->cap_window < g.W))
        return HYQ_ERR_INVALID_ARG;
    if (!need_pointers) return HYQ_OK;
    if (g.nQ > 0 && (!c->kq_codes || !c->vq_codes || !c->kq_scales || !c->vq_scales)) return HYQ_ERR_INVALID_ARG;
    if (c->k > 0 && (!c->k_vl || !c->v_vl)) return HYQ_ERR_INVALID_ARG;
    if (g.W > 0 && (!c->k_win || !c->v_win)) return HYQ_ERR_INVALID_ARG;
    if (c->n_staging > 0 && (!c->k_s || !c->v_s)) return HYQ_ERR_INVALID_ARG;
    const void* al[] = {c->kq_codes, c->vq_codes, c->k_vl, c->v_vl, c->k_win, c->v_win, c->k_s, c->v_s};
    for (const void* p : al)
        if (!aligned16(p)) return HYQ_ERR_ALIGNMENT;
    // the scales are read one float at a time (a sequence's slice of a batch allocation need not be 16-byte aligned)
    if ((reinterpret_cast<uintptr_t>(c->kq_scales) | reinterpret_cast<uintptr_t>(c->vq_scales)) & 3u) return HYQ_ERR_ALIGNMENT;
    return HYQ_OK;
}

extern "C" {

int hyq_kv_cache_query_sizes(const hyq_kv_cache* cache, hyq_kv_cache_sizes* sizes) {
    if (!sizes) return HYQ_ERR_INVALID_ARG;
    const int rc = check_cache(cache, false);
    if (rc != HYQ_OK) return rc;
    const CacheGeo g = cache_geo(*cache);
    const size_t heads = (size_t)cache->B * cache->Hkv;
    sizes->quantized_rows = g.nQ;
    sizes->padded_rows = g.nQp;
    const size_t row_bytes = cache->format == HYQ_FMT_INT4 ? HYQ_D / 2 : HYQ_D;
    sizes->kq_codes_bytes = heads * g.sQ * row_bytes;
    sizes->vq_codes_bytes = heads * g.sQ * row_bytes;
    sizes->scales_bytes = heads * (g.sQ / cache->group) * sizeof(float);
    sizes->vertical_bytes = heads * g.sK * HYQ_D * 2;
    sizes->window_bytes = heads * g.sW * HYQ_D * 2;
    sizes->staging_bytes = heads * cache->staging_capacity * HYQ_D * 2;
    return HYQ_OK;
}

int hyq_freeze(const void* k_, const void* v, const int32_t* vl_idx, const hyq_kv_cache* cache, void* stream) {
    const int rc = check_cache(cache, true);
    if (rc != HYQ_OK) return rc;
    if (!k_ || !v || (cache->k > 0 && !vl_idx)) return HYQ_ERR_INVALID_ARG;
    if (!aligned16(k_) || !aligned16(v) || (reinterpret_cast<uintptr_t>(vl_idx) & 3u)) return HYQ_ERR_ALIGNMENT;
    return launch_freeze(k_, v, vl_idx, *cache, static_cast<cudaStream_t>(stream));
}

int hyq_kv_cache_append(const void* k_new, const void* v_new, const hyq_kv_cache* cache, void* stream) {
    const int rc = check_cache(cache, false);
    if (rc != HYQ_OK) return rc;
    if (!k_new || !v_new || !cache->k_s || !cache->v_s || cache->n_staging >= cache->staging_capacity) return HYQ_ERR_INVALID_ARG;
    if (!aligned16(k_new) || !aligned16(v_new) || !aligned16(cache->k_s) || !aligned16(cache->v_s)) return HYQ_ERR_ALIGNMENT;
    return launch_cache_append(k_new, v_new, *cache, static_cast<cudaStream_t>(stream));
}

int hyq_hybrid_attention_decode_workspace(const hyq_kv_cache* cache, int splits, size_t* bytes) {
    if (!bytes || splits < 0 || splits > 1024) return HYQ_ERR_INVALID_ARG;
    const int rc = check_cache(cache, false);
    if (rc != HYQ_OK) return rc;
    *bytes = decode_workspace_bytes(*cache, splits > 0 ? splits : decode_auto_splits(*cache));
    return HYQ_OK;
}

int hyq_hybrid_attention_decode(const void* q, const hyq_kv_cache* cache, float softmax_scale, int splits, int out_dtype,
                                void* out, float* lse, void* workspace, size_t workspace_bytes, void* stream) {
    const int rc = check_cache(cache, true);
    if (rc != HYQ_OK) return rc;
    if (!q || !out || !workspace || splits < 0 || splits > 1024) return HYQ_ERR_INVALID_ARG;
    if (out_dtype != 0 && out_dtype != 1) return HYQ_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(out) || !aligned16(workspace)) return HYQ_ERR_ALIGNMENT;
    const int s = splits > 0 ? splits : decode_auto_splits(*cache);
    if (workspace_bytes < decode_workspace_bytes(*cache, s)) return HYQ_ERR_WORKSPACE;
    const float alpha = softmax_scale != 0.0f ? softmax_scale : 1.0f / std::sqrt((float)cache->D);
    return launch_decode(q, *cache, nullptr, alpha, s, out_dtype, out, lse, workspace, static_cast<cudaStream_t>(stream));
}

int hyq_hybrid_attention_decode_ragged(const void* q, const hyq_kv_cache* cache, const int32_t* lengths, float softmax_scale,
                                       int splits, int out_dtype, void* out, float* lse, void* workspace,
                                       size_t workspace_bytes, void* stream) {
    const int rc = check_cache(cache, true);
    if (rc != HYQ_OK) return rc;
    if (!q || !out || !workspace || !lengths || splits < 0 || splits > 1024) return HYQ_ERR_INVALID_ARG;
    if (out_dtype != 0 && out_dtype != 1) return HYQ_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(out) || !aligned16(workspace) || !aligned16(lengths)) return HYQ_ERR_ALIGNMENT;
    const int s = splits > 0 ? splits : decode_auto_splits(*cache);
    if (workspace_bytes < decode_workspace_bytes(*cache, s)) return HYQ_ERR_WORKSPACE;
    const float alpha = softmax_scale != 0.0f ? softmax_scale : 1.0f / std::sqrt((float)cache->D);
    return launch_decode(q, *cache, lengths, alpha, s, out_dtype, out, lse, workspace, static_cast<cudaStream_t>(stream));
}

}  // extern "C"
