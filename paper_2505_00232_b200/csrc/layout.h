// Packed weight layout shared by the host packer and the device kernels.
//
// The blob is a 256-byte header followed by the body and, for per-channel scales, a scale array.
// The body is ordered so that both kernels stream it front to back in large contiguous pieces
// (the idea of the paper's Section 3.1: store weights in the permutation the kernel reads):
//
//   for rsb in row super-blocks of 128 output channels        (the prefill kernel's tile height)
//     for kc in k-chunks (64 k for int4, 32 k for int8)
//       block(rsb, kc):
//         weights : 8 row-blocks x 32 lanes x 16 bytes = 4096 B
//         scales  : 8 row-blocks x 8 x 8 bytes = 512 B          (grouped int4 only)
//
// A row-block is 16 output channels.  Lane (g = lane / 4, c = lane % 4) of a row-block owns rows
// g and g + 8 and, per chunk, the k positions  8c .. 8c+7  (int8) or  8c .. 8c+7 and 32+8c .. 32+8c+7
// (int4): exactly the operand fragment of a 16x8x16 warp MMA, so the decode kernel feeds a 16-byte
// load straight to the tensor cores, and the prefill kernel turns the same 16 bytes into 16-byte
// runs of one row of its fp16 shared-memory tile.
//
// int4 word i (i = 0..3) of a lane covers k = 32*(i/2) + 8c + 4*(i%2) + j, j = 0..3, nibble p holding
//   p: 0      1        2      3        4      5        6      7
//      (g,j0) (g+8,j0) (g,j2) (g+8,j2) (g,j1) (g+8,j1) (g,j3) (g+8,j3)      stored as q + 8.
// int8 word w (w = 0..3) covers k = 8c + 4*(w/2) + 2*(w%2) + {0,1}, bytes
//      (g,ka) (g,kb) (g+8,ka) (g+8,kb)                                       stored as q + 128.
// Grouped scales of lane-row g in a block: 4 fp16 = s[g][G0] s[g][G1] s[g+8][G0] s[g+8][G1], G0/G1 the
// two 32-wide groups of the chunk (a coarser group size is expanded to 32 at pack time).
#pragma once
#include <stdint.h>
#include <stddef.h>

#ifndef QL_HD
#ifdef __CUDACC__
#define QL_HD __host__ __device__ __forceinline__
#else
#define QL_HD inline
#endif
#endif

namespace ql {

constexpr uint32_t kMagic = 0x31424C51u;   // "QLB1"
constexpr uint32_t kLayoutVersion = 1;
constexpr int kHeaderBytes = 256;
constexpr int kRsbRows = 128;              // rows per row super-block
constexpr int kRbRows = 16;                // rows per row-block (one warp-MMA tile)
constexpr int kWeightBlockBytes = 4096;    // 8 row-blocks x 32 lanes x 16 B
constexpr int kScaleBlockBytes = 512;      // 8 row-blocks x 8 g x 4 fp16

struct Layout {
    int32_t N, K, bits, group;
    int32_t grouped;          // 1: scales interleaved per block (int4 with group != 0)
    int32_t chunk_k;          // k per chunk: 64 (int4) or 32 (int8)
    int32_t n_rsb, n_kc;      // row super-blocks, k-chunks
    int32_t block_bytes;      // bytes of one (rsb, kc) block
    int64_t body_offset;      // from blob start
    int64_t chan_scale_offset;// from blob start; 0 if grouped
    int64_t total_bytes;
};

struct Header {               // first bytes of the blob; the rest of the 256 bytes is zero
    uint32_t magic, version;
    int32_t N, K, bits, group;
    int32_t chunk_k, block_bytes, n_rsb, n_kc;
    int64_t body_offset, chan_scale_offset, total_bytes;
};

// Returns false if the descriptor is invalid or unsupported.
inline bool make_layout(int32_t N, int32_t K, int32_t bits, int32_t group, Layout* L)
{
    if (N < 8 || K < 32 || (N % 8) || (K % 32)) return false;
    if (bits == 8) { if (group != 0) return false; }
    else if (bits == 4) { if (!(group == 0 || group == 32 || group == 64 || group == 128)) return false;
                          if (group && (K % group)) return false; }
    else return false;
    L->N = N; L->K = K; L->bits = bits; L->group = group;
    L->grouped = (bits == 4 && group != 0) ? 1 : 0;
    L->chunk_k = bits == 4 ? 64 : 32;
    L->n_rsb = (N + kRsbRows - 1) / kRsbRows;
    L->n_kc = (K + L->chunk_k - 1) / L->chunk_k;
    L->block_bytes = kWeightBlockBytes + (L->grouped ? kScaleBlockBytes : 0);
    L->body_offset = kHeaderBytes;
    int64_t body = (int64_t)L->n_rsb * L->n_kc * L->block_bytes;
    if (L->grouped) { L->chan_scale_offset = 0; L->total_bytes = L->body_offset + body; }
    else {
        L->chan_scale_offset = L->body_offset + body;               // multiple of 256
        int64_t sc = (int64_t)L->n_rsb * kRsbRows * 2;
        L->total_bytes = L->chan_scale_offset + ((sc + 255) / 256) * 256;
    }
    return true;
}

// k offset inside a chunk of (lane-column c, int4 word i, slot j)
QL_HD int int4_k_in_chunk(int c, int i, int j) { return 32 * (i >> 1) + 8 * c + 4 * (i & 1) + j; }
// (row select 0/1, slot j) held by nibble p of an int4 word
QL_HD int int4_nibble_rowsel(int p) { return p & 1; }
QL_HD int int4_nibble_slot(int p) { return ((p >> 1) & 1) * 2 + (p >> 2); }
// k offset inside a chunk of (lane-column c, int8 word w, byte b); row select of byte b
QL_HD int int8_k_in_chunk(int c, int w, int b) { return 8 * c + 4 * (w >> 1) + 2 * (w & 1) + (b & 1); }
QL_HD int int8_byte_rowsel(int b) { return b >> 1; }

}  // namespace ql
