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
    size_t vl_tiles;    // u8   [B*Hq][mask_words/2][2048]  FP8 / INT4 scores only: per 64-key tile a 64 x 32 e5m2 operand, -inf in
                        //                              element 0 of a vertical-line key's row, zero elsewhere (two 16-byte column
                        //                              chunks, each [64 keys][16 bytes])
    size_t redo;        // u32  [1 + 3 * CTAs]          block indices of the CTAs whose work the second launch does again, behind their count
    size_t part_o;      // f32  [splits][B*Hq][Lq][D]   split keys only: partial accumulators ...
    size_t part_ml;     // f32  [splits][B*Hq][Lq][2]   ... and (reference maximum, row sum) per row
    size_t total;
    int mask_words;     // words per head, a multiple of 4 (one 16-byte group per 128-key tile)
    int splits;         // CTAs per pair of query tiles (1: the keys are not split)
};

// Short query blocks leave most SMs without a CTA (one CTA per 256 query rows and head): the walk over the keys is
// then split over several CTAs.  Returns how many (1..8), so that the grid reaches about two CTAs per SM while
// every slice keeps a useful number of key tiles.
int tc_key_splits(const hyq_attn_args& a);

TcWorkspace tc_workspace_layout(const hyq_attn_args& a);
int launch_tc_prepass(const hyq_attn_args& a, const TcWorkspace& w, cudaStream_t st);

// Test hooks of the tensor-core kernel (hyq_test_set_attention_hooks): the clock limit of a single barrier wait
// (0: the default of about two seconds) and the walk position whose K/V load the producer leaves out (-1: none).
struct TcTestHooks {
    long long wait_limit;
    int drop_load;
};
TcTestHooks tc_test_hooks();

constexpr int VL_TILE_BYTES = 2048;

// zero-fills bits[n_heads][mask_words] and sets one bit per vertical-line key (memset + one kernel)
int launch_vl_bitmask(const int32_t* idx, long n_heads, int k, int L, int mask_words, uint32_t* bits, cudaStream_t st);

}  // namespace hyq
