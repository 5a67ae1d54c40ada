// Geometry of the hybrid KV cache shared by the Freeze and decode kernels (layout only).
#pragma once
#include "common.cuh"
#include "../../include/hyq_decode.h"

namespace hyq {

constexpr int DEC_TILE_KEYS = 16;          // rows per matrix-instruction tile
constexpr int DEC_VTILE_BYTES = 1024;      // 16 rows x 128 channels x 4 bits
constexpr int DEC_MAX_GROUP = 8;           // query heads per KV head (the n = 8 side of m16n8k16)

struct CacheGeo {
    int W;              // rows in the window buffers: min(window, N)
    long nQ, nQp;       // quantized rows per head: valid, padded to whole groups of G rows
    long sQ, sK, sW;    // rows between consecutive heads in the quantized, vertical and window buffers
};

static inline CacheGeo cache_geo(const hyq_kv_cache& c) {
    CacheGeo g;
    g.W = c.window < c.N ? c.window : c.N;
    g.nQ = (long)c.N - g.W - c.k;
    const long G = c.group > 0 ? c.group : 64;
    g.nQp = (g.nQ + G - 1) / G * G;
    g.sQ = c.cap_quantized_rows ? c.cap_quantized_rows : g.nQp;
    g.sK = c.cap_vertical ? c.cap_vertical : c.k;
    g.sW = c.cap_window ? c.cap_window : g.W;
    return g;
}

// Byte of a V tile that holds channels (d, d + 1), d even, of row `key` (0..15) of the tile: lane l = 4r + j
// owns words x = 0..3 at bytes [16l, 16l + 16) and words x = 4..7 at bytes [512 + 16l, 512 + 16l + 16); nibble n of
// word x of that lane is channel 64*(x>>2) + 8r + 2*(x&3) + (n&1) of row 2j + (n>>2) + 8*((n>>1)&1).
__host__ __device__ __forceinline__ int vq_byte_offset(int key, int d) {
    const int j = (key & 7) >> 1, n = ((key >> 3) << 1) | ((key & 1) << 2);
    const int r = (d >> 3) & 7, x = ((d >> 6) << 2) | ((d >> 1) & 3);
    return (x >> 2) * 512 + (4 * r + j) * 16 + (x & 3) * 4 + (n >> 1);
}

// Same for an INT8 V tile (2048 bytes): byte of channel d of row `key`.  Lane l = 4r + j owns bytes [16l, 16l + 16) of
// each of the tile's four 512-byte runs, 16 words in all; word 2x + (key >> 3) holds, in byte order, (channel e = 0,
// key bit 0 = 0), (e = 0, 1), (e = 1, 0), (e = 1, 1) of accumulator row pair x - so a byte permute picks the two
// key-adjacent codes of an operand register.
__host__ __device__ __forceinline__ int vq8_byte_offset(int key, int d) {
    const int j = (key & 7) >> 1, r = (d >> 3) & 7, x = ((d >> 6) << 2) | ((d >> 1) & 3);
    const int w = 2 * x + (key >> 3);
    return (w >> 2) * 512 + (4 * r + j) * 16 + (w & 3) * 4 + (d & 1) * 2 + (key & 1);
}

int launch_freeze(const void* k_, const void* v, const int32_t* vl_idx, const hyq_kv_cache& c, cudaStream_t st);
int launch_cache_append(const void* k_new, const void* v_new, const hyq_kv_cache& c, cudaStream_t st);
int decode_auto_splits(const hyq_kv_cache& c);
size_t decode_workspace_bytes(const hyq_kv_cache& c, int splits);
int launch_decode(const void* q, const hyq_kv_cache& c, const int32_t* lengths, float alpha, int splits, int out_dtype,
                  void* out, float* lse, void* workspace, cudaStream_t st);

}  // namespace hyq
