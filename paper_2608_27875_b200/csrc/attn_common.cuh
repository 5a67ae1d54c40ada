// Declarations shared by the attention pre-pass and the attention kernels.
#pragma once
#include "common.cuh"

namespace hyq {

// number of query rows of a call (the query block may be shorter than the keys; 0 means "all L")
__host__ __device__ inline int query_rows(const hyq_attn_args& a) { return a.Lq > 0 ? a.Lq : a.L; }

// byte offsets into the caller's workspace (tensor-core kernel)
struct TcWorkspace {
    size_t vl_bits;     // uint32 [B*Hq][mask_words]   vertical-line bitmask over key positions
    size_t v16;         // fp16 [B*Hkv][L][D]           V
    size_t vh16;        // fp16 [B*Hkv][L][D]           V^ = code * scale
    size_t kvl;         // bf16 [B*Hq][k][D]            gathered vertical-line K rows
    size_t vvl;         // fp16 [B*Hq][k][D]            gathered vertical-line V rows
    size_t q8;          // u8   [B*Hq][Lq][D]           INT4 only: Q codes as e4m3 bytes
    size_t k8;          // u8   [B*Hkv][L][D]           INT4 only: K codes as e4m3 bytes
    size_t total;
    int mask_words;
};

TcWorkspace tc_workspace_layout(const hyq_attn_args& a);
int launch_tc_prepass(const hyq_attn_args& a, const TcWorkspace& w, cudaStream_t st);

// zero-fills bits[n_heads][mask_words] and sets one bit per vertical-line key (memset + one kernel)
int launch_vl_bitmask(const int32_t* idx, long n_heads, int k, int L, int mask_words, uint32_t* bits, cudaStream_t st);

}  // namespace hyq
