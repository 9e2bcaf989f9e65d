// Host-side weights conversion (paper Section 3.4 "weights conversion", Section 3.1 weight layouts):
// canonical integers + fp16 scales  <->  the tile-ordered blob described in layout.h.
// Pure host code, integer shuffles only; calls no CUDA.
#include <cstring>
#include <vector>

#include "../../include/qlinear.h"
#include "layout.h"

using namespace ql;

namespace {

inline int64_t block_offset(const Layout& L, int rsb, int kc)
{
    return L.body_offset + ((int64_t)rsb * L.n_kc + kc) * L.block_bytes;
}

// original scale-group index of column k
inline int group_of(const Layout& L, int k) { return L.group ? k / L.group : 0; }
inline int n_groups(const Layout& L) { return L.group ? L.K / L.group : 1; }

}  // namespace

extern "C" size_t qlinear_packed_size(const qlinear_desc* d)
{
    Layout L;
    if (!d || !make_layout(d->N, d->K, d->bits, d->group, &L)) return 0;
    return (size_t)L.total_bytes;
}

extern "C" ql_status qlinear_pack(const qlinear_desc* d, const int8_t* q, const uint16_t* s,
                                  void* packed, size_t packed_bytes)
{
    if (!d || !q || !s || !packed) return QL_ERR_INVALID_ARG;
    Layout L;
    if (!make_layout(d->N, d->K, d->bits, d->group, &L)) return QL_ERR_UNSUPPORTED;
    if (packed_bytes < (size_t)L.total_bytes) return QL_ERR_INVALID_ARG;
    const int N = L.N, K = L.K;
    if (L.bits == 4) {
        for (int64_t i = 0, e = (int64_t)N * K; i < e; ++i)
            if (q[i] < -8 || q[i] > 7) return QL_ERR_INVALID_ARG;
    }
    uint8_t* out = static_cast<uint8_t*>(packed);
    std::memset(out, 0, (size_t)L.total_bytes);
    Header h{};
    h.magic = kMagic; h.version = kLayoutVersion;
    h.N = N; h.K = K; h.bits = L.bits; h.group = L.group;
    h.chunk_k = L.chunk_k; h.block_bytes = L.block_bytes; h.n_rsb = L.n_rsb; h.n_kc = L.n_kc;
    h.body_offset = L.body_offset; h.chan_scale_offset = L.chan_scale_offset; h.total_bytes = L.total_bytes;
    std::memcpy(out, &h, sizeof(h));

    const int ng = n_groups(L);
    auto qv = [&](int row, int k) -> int { return (row < N && k < K) ? q[(int64_t)row * K + k] : 0; };

    for (int rsb = 0; rsb < L.n_rsb; ++rsb)
        for (int kc = 0; kc < L.n_kc; ++kc) {
            uint8_t* blk = out + block_offset(L, rsb, kc);
            for (int rb = 0; rb < 8; ++rb)
                for (int lane = 0; lane < 32; ++lane) {
                    const int g = lane >> 2, c = lane & 3;
                    const int row0 = rsb * kRsbRows + rb * kRbRows + g;
                    uint32_t words[4];
                    if (L.bits == 4) {
                        for (int i = 0; i < 4; ++i) {
                            uint32_t w = 0;
                            for (int p = 0; p < 8; ++p) {
                                int row = row0 + 8 * int4_nibble_rowsel(p);
                                int k = kc * 64 + int4_k_in_chunk(c, i, int4_nibble_slot(p));
                                w |= (uint32_t)((qv(row, k) + 8) & 0xF) << (4 * p);
                            }
                            words[i] = w;
                        }
                    } else {
                        for (int wi = 0; wi < 4; ++wi) {
                            uint32_t w = 0;
                            for (int b = 0; b < 4; ++b) {
                                int row = row0 + 8 * int8_byte_rowsel(b);
                                int k = kc * 32 + int8_k_in_chunk(c, wi, b);
                                w |= (uint32_t)((qv(row, k) + 128) & 0xFF) << (8 * b);
                            }
                            words[wi] = w;
                        }
                    }
                    std::memcpy(blk + rb * 512 + lane * 16, words, 16);
                }
            if (L.grouped) {
                uint16_t* sc = reinterpret_cast<uint16_t*>(blk + kWeightBlockBytes);
                for (int rb = 0; rb < 8; ++rb)
                    for (int g = 0; g < 8; ++g)
                        for (int rs = 0; rs < 2; ++rs)
                            for (int hg = 0; hg < 2; ++hg) {
                                int row = rsb * kRsbRows + rb * kRbRows + g + 8 * rs;
                                int k = kc * 64 + 32 * hg;
                                uint16_t v = (row < N && k < K) ? s[(int64_t)row * ng + group_of(L, k)] : 0;
                                sc[(rb * 8 + g) * 4 + rs * 2 + hg] = v;
                            }
            }
        }
    if (!L.grouped) {
        uint16_t* sc = reinterpret_cast<uint16_t*>(out + L.chan_scale_offset);
        for (int n = 0; n < N; ++n) sc[n] = s[n];
    }
    return QL_OK;
}

extern "C" ql_status qlinear_unpack(const qlinear_desc* d, const void* packed, int8_t* q_out, uint16_t* s_out)
{
    if (!d || !packed || !q_out || !s_out) return QL_ERR_INVALID_ARG;
    Layout L;
    if (!make_layout(d->N, d->K, d->bits, d->group, &L)) return QL_ERR_UNSUPPORTED;
    const uint8_t* in = static_cast<const uint8_t*>(packed);
    Header h;
    std::memcpy(&h, in, sizeof(h));
    if (h.magic != kMagic || h.version != kLayoutVersion || h.N != L.N || h.K != L.K || h.bits != L.bits ||
        h.group != L.group || h.total_bytes != L.total_bytes)
        return QL_ERR_INVALID_ARG;
    const int N = L.N, K = L.K, ng = n_groups(L);
    for (int rsb = 0; rsb < L.n_rsb; ++rsb)
        for (int kc = 0; kc < L.n_kc; ++kc) {
            const uint8_t* blk = in + block_offset(L, rsb, kc);
            for (int rb = 0; rb < 8; ++rb)
                for (int lane = 0; lane < 32; ++lane) {
                    const int g = lane >> 2, c = lane & 3;
                    const int row0 = rsb * kRsbRows + rb * kRbRows + g;
                    uint32_t words[4];
                    std::memcpy(words, blk + rb * 512 + lane * 16, 16);
                    if (L.bits == 4) {
                        for (int i = 0; i < 4; ++i)
                            for (int p = 0; p < 8; ++p) {
                                int row = row0 + 8 * int4_nibble_rowsel(p);
                                int k = kc * 64 + int4_k_in_chunk(c, i, int4_nibble_slot(p));
                                if (row < N && k < K)
                                    q_out[(int64_t)row * K + k] = (int8_t)((int)((words[i] >> (4 * p)) & 0xF) - 8);
                            }
                    } else {
                        for (int wi = 0; wi < 4; ++wi)
                            for (int b = 0; b < 4; ++b) {
                                int row = row0 + 8 * int8_byte_rowsel(b);
                                int k = kc * 32 + int8_k_in_chunk(c, wi, b);
                                if (row < N && k < K)
                                    q_out[(int64_t)row * K + k] = (int8_t)((int)((words[wi] >> (8 * b)) & 0xFF) - 128);
                            }
                    }
                }
            if (L.grouped) {
                const uint16_t* sc = reinterpret_cast<const uint16_t*>(blk + kWeightBlockBytes);
                for (int rb = 0; rb < 8; ++rb)
                    for (int g = 0; g < 8; ++g)
                        for (int rs = 0; rs < 2; ++rs)
                            for (int hg = 0; hg < 2; ++hg) {
                                int row = rsb * kRsbRows + rb * kRbRows + g + 8 * rs;
                                int k = kc * 64 + 32 * hg;
                                if (row < N && k < K && (k % L.group) == 0)
                                    s_out[(int64_t)row * ng + k / L.group] = sc[(rb * 8 + g) * 4 + rs * 2 + hg];
                            }
            }
        }
    if (!L.grouped) {
        const uint16_t* sc = reinterpret_cast<const uint16_t*>(in + L.chan_scale_offset);
        for (int n = 0; n < N; ++n) s_out[n] = sc[n];
    }
    return QL_OK;
}
