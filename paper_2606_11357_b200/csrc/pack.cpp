// Host-side offline pre-tiling (Section 4.2 of the paper): AWQ / int8 weights -> packed blob.
// Pure byte shuffling; scales are copied bit for bit.
#include <string.h>

#include "../../include/tilefuse.h"
#include "layout.h"

namespace {

constexpr int kAwqPosOfColumn[8] = {0, 4, 1, 5, 2, 6, 3, 7};   // nibble position of column c%8

inline uint32_t awq_code(const uint32_t* words, size_t row_words, int r, int c) {
    return (words[(size_t)r * row_words + (c >> 3)] >> (4 * kAwqPosOfColumn[c & 7])) & 0xFu;
}

bool legal_shape(int bits, int K, int N, int g) {
    if (bits != 4 && bits != 8) return false;
    if (K < tf::kTileK || K > TF_MAX_DIM || N < 8 || N > TF_MAX_DIM) return false;
    if (N % 8 != 0) return false;
    if (g <= 0 || K % g != 0) return false;
    if (g % tf::kTileK == 0) return true;
    return bits == 4 && (g == 64 || g == 32);      // several groups inside a tile: the 4-bit format only
}

void write_header(void* out, int bits, int K, int N, int g, size_t total) {
    tf_blob_header h;
    memset(&h, 0, sizeof(h));
    h.magic = tf::kMagic;
    h.version = tf::kBlobVersion;
    h.bits = (uint32_t)bits;
    h.K = (uint32_t)K;
    h.N = (uint32_t)N;
    h.group_size = (uint32_t)g;
    h.n_padded = (uint32_t)((N + tf::kTileN - 1) / tf::kTileN * tf::kTileN);
    h.strips = h.n_padded / tf::kTileN;
    h.ktiles = (uint32_t)(K / tf::kTileK);
    h.tile_bytes = (uint32_t)tf::tile_bytes(bits, tf::groups_per_tile(g));
    h.tiles_offset = tf::kHeaderBytes;
    h.total_bytes = total;
    memcpy(out, &h, sizeof(h));
}

// Physical (k, n) offsets inside a tile of register `reg` (0..3), element `el` (0..1) of
// lane (g, t) in k-block kb, n-block w.
inline void tile_coord(int kb, int g, int t, int w, int reg, int el, int* dk, int* dn) {
    *dk = 16 * kb + 4 * t + 2 * (reg >> 1) + el;
    *dn = 16 * w + g + 8 * (reg & 1);
}

void write_scales(uint8_t* tile_scales, const uint16_t* scales, int N, int grp, int n0) {
    uint16_t* s = reinterpret_cast<uint16_t*>(tile_scales);
    for (int g = 0; g < 8; ++g)
        for (int w = 0; w < 4; ++w)
            for (int h = 0; h < 2; ++h) {
                int n = n0 + 16 * w + g + 8 * h;
                s[g * 8 + 2 * w + h] = n < N ? scales[(size_t)grp * N + n] : (uint16_t)0;
            }
}

}  // namespace

static_assert(sizeof(tf_blob_header) == tf::kHeaderBytes, "header must be 256 bytes");

extern "C" __attribute__((visibility("default"))) size_t tf_packed_size(int bits, int K, int N, int group_size) {
    if (!legal_shape(bits, K, N, group_size)) return 0;
    size_t strips = (size_t)(N + tf::kTileN - 1) / tf::kTileN;
    size_t ktiles = (size_t)K / tf::kTileK;
    size_t tile = (size_t)tf::tile_bytes(bits, tf::groups_per_tile(group_size));
    return tf::kHeaderBytes + strips * ktiles * tile;
}

extern "C" __attribute__((visibility("default"))) tf_status tf_pack_awq(const uint32_t* qweight, const uint16_t* scales_fp16,
                                 const uint32_t* qzeros, int K, int N, int group_size,
                                 void* out, size_t out_bytes) {
    if (!qweight || !scales_fp16 || !qzeros || !out) return TF_ERR_NULL;
    size_t total = tf_packed_size(4, K, N, group_size);
    if (total == 0) return TF_ERR_SHAPE;
    if (out_bytes < total) return TF_ERR_WORKSPACE;
    write_header(out, 4, K, N, group_size, total);
    const size_t row_words = (size_t)N / 8;
    const int strips = (N + tf::kTileN - 1) / tf::kTileN, ktiles = K / tf::kTileK;
    uint8_t* base = static_cast<uint8_t*>(out) + tf::kHeaderBytes;
    const int G = tf::groups_per_tile(group_size), tile_bytes = tf::w4_tile_bytes(G);
    for (int S = 0; S < strips; ++S) {
        const int n0 = S * tf::kTileN;
        for (int T = 0; T < ktiles; ++T) {
            const int k0 = T * tf::kTileK;
            uint8_t* tile = base + ((size_t)S * ktiles + T) * tile_bytes;
            uint32_t* wq = reinterpret_cast<uint32_t*>(tile);
            for (int kb = 0; kb < 8; ++kb)
                for (int lane = 0; lane < 32; ++lane)
                    for (int w = 0; w < 4; ++w) {
                        const int g = lane >> 2, t = lane & 3;
                        uint32_t word = 0;
                        for (int p = 0; p < 8; ++p) {
                            int dk, dn;
                            tile_coord(kb, g, t, w, p & 3, p >> 2, &dk, &dn);
                            const int n = n0 + dn;
                            // padded columns: q = z = 0, s = 0  ->  dequantizes to exactly 0
                            uint32_t code = n < N ? awq_code(qweight, row_words, k0 + dk, n) : 0u;
                            word |= code << (4 * p);
                        }
                        wq[(kb * 32 + lane) * 4 + w] = word;
                    }
            for (int gr = 0; gr < G; ++gr) {                 // the groups that meet this tile, along k
                const int grp = (k0 + gr * (tf::kTileK / G)) / group_size;
                write_scales(tile + tf::w4_scale_offset(gr), scales_fp16, N, grp, n0);
                uint32_t* zq = reinterpret_cast<uint32_t*>(tile + tf::w4_zero_offset(G, gr));
                for (int g = 0; g < 8; ++g) {
                    uint32_t word = 0;
                    for (int i = 0; i < 8; ++i) {
                        const int n = n0 + 16 * (i & 3) + g + 8 * (i >> 2);
                        uint32_t code = n < N ? awq_code(qzeros, row_words, grp, n) : 0u;
                        word |= code << (4 * i);
                    }
                    zq[g] = word;
                }
            }
        }
    }
    return TF_OK;
}

extern "C" __attribute__((visibility("default"))) tf_status tf_pack_w8(const int8_t* w8, const uint16_t* scales_fp16, int K, int N,
                                int group_size, void* out, size_t out_bytes) {
    if (!w8 || !scales_fp16 || !out) return TF_ERR_NULL;
    size_t total = tf_packed_size(8, K, N, group_size);
    if (total == 0) return TF_ERR_SHAPE;
    if (out_bytes < total) return TF_ERR_WORKSPACE;
    write_header(out, 8, K, N, group_size, total);
    const int strips = (N + tf::kTileN - 1) / tf::kTileN, ktiles = K / tf::kTileK;
    uint8_t* base = static_cast<uint8_t*>(out) + tf::kHeaderBytes;
    for (int S = 0; S < strips; ++S) {
        const int n0 = S * tf::kTileN;
        for (int T = 0; T < ktiles; ++T) {
            const int k0 = T * tf::kTileK, grp = k0 / group_size;
            uint8_t* tile = base + ((size_t)S * ktiles + T) * tf::kW8TileBytes;
            for (int kb = 0; kb < 8; ++kb)
                for (int lane = 0; lane < 32; ++lane)
                    for (int w = 0; w < 4; ++w)
                        for (int r = 0; r < 2; ++r) {
                            const int g = lane >> 2, t = lane & 3;
                            uint8_t* dst = tile + (((size_t)(kb * 2 + (w >> 1)) * 32 + lane) * 4 +
                                                   2 * (w & 1) + r) * 4;
                            for (int b = 0; b < 4; ++b) {
                                int dk, dn;
                                tile_coord(kb, g, t, w, 2 * r + (b >> 1), b & 1, &dk, &dn);
                                const int n = n0 + dn;
                                dst[b] = n < N ? (uint8_t)w8[(size_t)(k0 + dk) * N + n] : (uint8_t)0;
                            }
                        }
            write_scales(tile + tf::kW8WeightBytes, scales_fp16, N, grp, n0);
        }
    }
    return TF_OK;
}

// Concatenation along N of blobs that share bits, K and group size (fused QKV, fused gate + up).  Section 4.5
// names the cost of dispatching many short GEMV operators per token; fewer, wider operators is the remedy at pack time.  Tiles are stored strip after strip, so the tiles
// of a part whose N is a multiple of the strip width are moved as they are; only the header changes.
extern "C" __attribute__((visibility("default"))) tf_status tf_pack_concat(const void* const* parts, int count, void* out,
                                                                           size_t out_bytes) {
    if (!parts || !out) return TF_ERR_NULL;
    if (count < 1) return TF_ERR_SHAPE;
    tf_blob_header first;
    long long n_total = 0;
    for (int i = 0; i < count; ++i) {
        if (!parts[i]) return TF_ERR_NULL;
        tf_blob_header h;
        memcpy(&h, parts[i], sizeof(h));
        if (h.magic != tf::kMagic || h.version != tf::kBlobVersion) return TF_ERR_BLOB;
        if (h.total_bytes != tf_packed_size((int)h.bits, (int)h.K, (int)h.N, (int)h.group_size) || h.total_bytes == 0)
            return TF_ERR_BLOB;
        if (i == 0) first = h;
        else if (h.bits != first.bits || h.K != first.K || h.group_size != first.group_size) return TF_ERR_SHAPE;
        if (i + 1 < count && h.N % tf::kTileN != 0) return TF_ERR_SHAPE;   // a part that is not last must end on a strip
        n_total += h.N;
    }
    if (n_total > TF_MAX_DIM) return TF_ERR_SHAPE;
    const size_t total = tf_packed_size((int)first.bits, (int)first.K, (int)n_total, (int)first.group_size);
    if (total == 0) return TF_ERR_SHAPE;
    if (out_bytes < total) return TF_ERR_WORKSPACE;
    uint8_t* dst = static_cast<uint8_t*>(out) + tf::kHeaderBytes;
    for (int i = 0; i < count; ++i) {
        tf_blob_header h;
        memcpy(&h, parts[i], sizeof(h));
        const size_t payload = (size_t)h.total_bytes - tf::kHeaderBytes;
        memcpy(dst, static_cast<const uint8_t*>(parts[i]) + tf::kHeaderBytes, payload);
        dst += payload;
    }
    write_header(out, (int)first.bits, (int)first.K, (int)n_total, (int)first.group_size, total);
    return TF_OK;
}

// Column-parallel sharding (Section 4.4: every worker owns distinct output columns, the activation vector is shared,
// no partial sums travel between workers).  Tiles are stored strip after strip, so the blob of a column range that
// starts and ends on strip boundaries is a contiguous byte range of the full blob plus a header of its own.
extern "C" __attribute__((visibility("default"))) tf_status tf_shard_columns(int N, int part, int parts, int* n_begin, int* n_count) {
    if (!n_begin || !n_count) return TF_ERR_NULL;
    if (N < 8 || N > TF_MAX_DIM || N % 8 != 0 || parts < 1 || part < 0 || part >= parts) return TF_ERR_SHAPE;
    const int strips = (N + tf::kTileN - 1) / tf::kTileN;
    if (parts > strips) return TF_ERR_SHAPE;                       // every part must own at least one strip
    const int s0 = (int)(((long long)part * strips) / parts), s1 = (int)(((long long)(part + 1) * strips) / parts);
    const int b = s0 * tf::kTileN, e = s1 * tf::kTileN < N ? s1 * tf::kTileN : N;
    *n_begin = b;
    *n_count = e - b;
    return TF_OK;
}

extern "C" __attribute__((visibility("default"))) tf_status tf_pack_shard(const void* packed, int part, int parts, void* out, size_t out_bytes) {
    if (!packed || !out) return TF_ERR_NULL;
    tf_blob_header h;
    memcpy(&h, packed, sizeof(h));
    if (h.magic != tf::kMagic || h.version != tf::kBlobVersion) return TF_ERR_BLOB;
    if (h.total_bytes == 0 || h.total_bytes != tf_packed_size((int)h.bits, (int)h.K, (int)h.N, (int)h.group_size)) return TF_ERR_BLOB;
    int n0 = 0, nc = 0;
    tf_status st = tf_shard_columns((int)h.N, part, parts, &n0, &nc);
    if (st != TF_OK) return st;
    const size_t total = tf_packed_size((int)h.bits, (int)h.K, nc, (int)h.group_size);
    if (total == 0) return TF_ERR_SHAPE;
    if (out_bytes < total) return TF_ERR_WORKSPACE;
    const size_t strip_bytes = (size_t)h.ktiles * h.tile_bytes;
    memcpy(static_cast<uint8_t*>(out) + tf::kHeaderBytes,
           static_cast<const uint8_t*>(packed) + tf::kHeaderBytes + (size_t)(n0 / tf::kTileN) * strip_bytes, total - tf::kHeaderBytes);
    write_header(out, (int)h.bits, (int)h.K, nc, (int)h.group_size, total);
    return TF_OK;
}
