// The tensor-core attention kernels compiled a second time, into namespace hyq::tcbt, with the quantization block
// size (32 or 128 tokens) as a run-time parameter; see the note at the top of attn_tc.cu.
#define HYQ_TC_VARIANT_BT 1
#include "attn_tc.cu"
