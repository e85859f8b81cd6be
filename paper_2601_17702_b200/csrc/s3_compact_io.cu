// Compact index on disk: host-side save / load of the per-layer arrays of the compact inverted index, with a
// checksum per layer and a structural check at load, so that a damaged file is refused instead of handing the
// scoring kernel offsets that leave its arrays. Plain host code; nothing here touches a device.
//
// File: 32-byte header {magic[8], u32 version, u32 n_layers, u32 d_sae, u32 0, u64 0}, then per layer a 32-byte record
// {u64 n_blocks, u64 n_words, u64 checksum, u64 0}, then per layer its arrays, each padded to 8 bytes: row_ptr
// (d_sae+1 u64), blk_ptr (d_sae+1 u32), blk_first (n_blocks i32), blk_desc (n_blocks u64), payload (n_words u32).
// Little-endian, as the arrays lie in memory.
#include <stdio.h>
#include <string.h>

#include <memory>

#include "s3_common.cuh"

namespace s3 {

namespace {

const char kMagic[8] = {'S', '3', 'C', 'I', 'D', 'X', 0, 1};
constexpr uint32_t kVersion = 1;

struct FileHeader {
    char magic[8];
    uint32_t version, n_layers, d_sae, zero0;
    uint64_t zero1;
};
struct LayerRecord {
    uint64_t n_blocks, n_words, checksum, zero;
};
static_assert(sizeof(FileHeader) == 32 && sizeof(LayerRecord) == 32, "file records are 32 bytes");

struct FileCloser {
    void operator()(FILE* f) const { if (f) fclose(f); }
};
using File = std::unique_ptr<FILE, FileCloser>;

uint64_t fnv1a(uint64_t h, const void* data, size_t n)
{
    const unsigned char* p = static_cast<const unsigned char*>(data);
    for (size_t i = 0; i < n; ++i) { h ^= p[i]; h *= 1099511628211ull; }
    return h;
}

uint64_t layer_checksum(const s3_compact_host_layer& L, int d_sae)
{
    uint64_t h = 14695981039346656037ull;
    h = fnv1a(h, L.h_row_ptr, (static_cast<size_t>(d_sae) + 1) * 8);
    h = fnv1a(h, L.h_blk_ptr, (static_cast<size_t>(d_sae) + 1) * 4);
    h = fnv1a(h, L.h_blk_first, L.n_blocks * 4);
    h = fnv1a(h, L.h_blk_desc, L.n_blocks * 8);
    h = fnv1a(h, L.h_payload, L.n_words * 4);
    return h;
}

// Every offset the scoring kernel derives from these arrays stays inside them.
s3_status check_layer(const s3_compact_host_layer& L, int d_sae, int layer)
{
    S3_REQUIRE(L.n_words >= 1 && L.h_payload[L.n_words - 1] == 0, S3_ERR_INVALID_ARG, "layer %d: payload lacks its closing zero word", layer);
    S3_REQUIRE(L.h_row_ptr[0] == 0 && L.h_blk_ptr[0] == 0, S3_ERR_INVALID_ARG, "layer %d: prefix arrays do not start at 0", layer);
    for (int f = 0; f < d_sae; ++f) {
        S3_REQUIRE(L.h_row_ptr[f + 1] >= L.h_row_ptr[f], S3_ERR_INVALID_ARG, "layer %d: row_ptr decreases at feature %d", layer, f);
        const uint64_t len = L.h_row_ptr[f + 1] - L.h_row_ptr[f];
        S3_REQUIRE(len <= 0x7FFFFFFFull, S3_ERR_INVALID_ARG, "layer %d: list of feature %d is longer than 2^31", layer, f);
        const uint64_t blocks = (len + 31) / 32;
        S3_REQUIRE(L.h_blk_ptr[f + 1] >= L.h_blk_ptr[f] && L.h_blk_ptr[f + 1] - L.h_blk_ptr[f] == blocks, S3_ERR_INVALID_ARG,
                   "layer %d: feature %d has %llu postings but its block range does not hold %llu blocks", layer, f,
                   (unsigned long long)len, (unsigned long long)blocks);
        for (uint64_t j = 0; j < blocks; ++j) {
            const uint64_t b = L.h_blk_ptr[f] + j;
            S3_REQUIRE(b < L.n_blocks, S3_ERR_INVALID_ARG, "layer %d: block index beyond n_blocks", layer);
            const uint64_t cnt = len - 32 * j < 32 ? len - 32 * j : 32;
            const uint64_t width = L.h_blk_desc[b] & 63u, off = L.h_blk_desc[b] >> 6;
            S3_REQUIRE(width <= 31, S3_ERR_INVALID_ARG, "layer %d: block %llu has width %llu", layer, (unsigned long long)b,
                       (unsigned long long)width);
            S3_REQUIRE(off + ((cnt - 1) * width + 31) / 32 <= L.n_words - 1, S3_ERR_INVALID_ARG,
                       "layer %d: block %llu reaches beyond the payload", layer, (unsigned long long)b);
            S3_REQUIRE(L.h_blk_first[b] >= 0, S3_ERR_INVALID_ARG, "layer %d: block %llu starts at a negative position", layer,
                       (unsigned long long)b);
        }
    }
    S3_REQUIRE(L.h_blk_ptr[d_sae] == L.n_blocks, S3_ERR_INVALID_ARG, "layer %d: blk_ptr ends at %u, n_blocks is %llu", layer,
               L.h_blk_ptr[d_sae], (unsigned long long)L.n_blocks);
    return S3_OK;
}

bool put(FILE* f, const void* p, size_t bytes)
{
    static const char pad[8] = {};
    if (bytes && fwrite(p, 1, bytes, f) != bytes) return false;
    const size_t r = (8 - bytes % 8) % 8;
    return r == 0 || fwrite(pad, 1, r, f) == r;
}

bool get(FILE* f, void* p, size_t bytes)
{
    char pad[8];
    if (bytes && fread(p, 1, bytes, f) != bytes) return false;
    const size_t r = (8 - bytes % 8) % 8;
    return r == 0 || fread(pad, 1, r, f) == r;
}

s3_status read_header(FILE* f, const char* path, FileHeader* h, LayerRecord* recs, int cap)
{
    S3_REQUIRE(fread(h, sizeof(*h), 1, f) == 1, S3_ERR_INVALID_ARG, "%s: shorter than a header", path);
    S3_REQUIRE(memcmp(h->magic, kMagic, 8) == 0, S3_ERR_INVALID_ARG, "%s: not a compact index file", path);
    S3_REQUIRE(h->version == kVersion, S3_ERR_UNSUPPORTED, "%s: file version %u, this library reads %u", path, h->version, kVersion);
    S3_REQUIRE(h->n_layers >= 1 && h->n_layers <= S3_MAX_SCORE_LAYERS && h->d_sae >= 1 && h->d_sae <= (1u << 20), S3_ERR_INVALID_ARG,
               "%s: n_layers = %u or d_sae = %u out of range", path, h->n_layers, h->d_sae);
    for (uint32_t l = 0; l < h->n_layers; ++l) {
        LayerRecord r;
        S3_REQUIRE(fread(&r, sizeof(r), 1, f) == 1, S3_ERR_INVALID_ARG, "%s: layer table cut short", path);
        if (static_cast<int>(l) < cap) recs[l] = r;
    }
    return S3_OK;
}

}  // namespace

}  // namespace s3

using namespace s3;

extern "C" {

s3_status s3_compact_save(const char* path, int n_layers, int d_sae, const s3_compact_host_layer* h_layers)
{
    S3_REQUIRE(path && h_layers, S3_ERR_INVALID_ARG, "null argument");
    S3_REQUIRE(n_layers >= 1 && n_layers <= S3_MAX_SCORE_LAYERS, S3_ERR_UNSUPPORTED, "n_layers = %d out of [1, %d]", n_layers,
               S3_MAX_SCORE_LAYERS);
    S3_REQUIRE(d_sae >= 1 && d_sae <= (1 << 20), S3_ERR_INVALID_ARG, "d_sae = %d out of range", d_sae);
    for (int l = 0; l < n_layers; ++l) {
        const s3_compact_host_layer& L = h_layers[l];
        S3_REQUIRE(L.h_row_ptr && L.h_blk_ptr && L.h_payload && ((L.h_blk_first && L.h_blk_desc) || L.n_blocks == 0), S3_ERR_INVALID_ARG,
                   "layer %d: null array", l);
        const s3_status st = check_layer(L, d_sae, l);
        if (st != S3_OK) return st;
    }
    File f(fopen(path, "wb"));
    S3_REQUIRE(f != nullptr, S3_ERR_STATE, "cannot open %s for writing", path);
    FileHeader h = {};
    memcpy(h.magic, kMagic, 8);
    h.version = kVersion; h.n_layers = static_cast<uint32_t>(n_layers); h.d_sae = static_cast<uint32_t>(d_sae);
    bool ok = fwrite(&h, sizeof(h), 1, f.get()) == 1;
    for (int l = 0; ok && l < n_layers; ++l) {
        LayerRecord r = {h_layers[l].n_blocks, h_layers[l].n_words, layer_checksum(h_layers[l], d_sae), 0};
        ok = fwrite(&r, sizeof(r), 1, f.get()) == 1;
    }
    for (int l = 0; ok && l < n_layers; ++l) {
        const s3_compact_host_layer& L = h_layers[l];
        ok = put(f.get(), L.h_row_ptr, (static_cast<size_t>(d_sae) + 1) * 8) && put(f.get(), L.h_blk_ptr, (static_cast<size_t>(d_sae) + 1) * 4) &&
             put(f.get(), L.h_blk_first, L.n_blocks * 4) && put(f.get(), L.h_blk_desc, L.n_blocks * 8) &&
             put(f.get(), L.h_payload, L.n_words * 4);
    }
    ok = ok && fflush(f.get()) == 0;
    S3_REQUIRE(ok, S3_ERR_STATE, "write to %s failed", path);
    return S3_OK;
}

s3_status s3_compact_file_info(const char* path, int* n_layers, int* d_sae, uint64_t* h_n_blocks, uint64_t* h_n_words, int cap_layers)
{
    S3_REQUIRE(path && n_layers && d_sae, S3_ERR_INVALID_ARG, "null argument");
    S3_REQUIRE(cap_layers >= 0 && (cap_layers == 0 || (h_n_blocks && h_n_words)), S3_ERR_INVALID_ARG, "null size arrays");
    File f(fopen(path, "rb"));
    S3_REQUIRE(f != nullptr, S3_ERR_STATE, "cannot open %s", path);
    FileHeader h;
    LayerRecord recs[S3_MAX_SCORE_LAYERS];
    const s3_status st = read_header(f.get(), path, &h, recs, S3_MAX_SCORE_LAYERS);
    if (st != S3_OK) return st;
    *n_layers = static_cast<int>(h.n_layers);
    *d_sae = static_cast<int>(h.d_sae);
    for (int l = 0; l < cap_layers && l < static_cast<int>(h.n_layers); ++l) {
        h_n_blocks[l] = recs[l].n_blocks;
        h_n_words[l] = recs[l].n_words;
    }
    return S3_OK;
}

s3_status s3_compact_load(const char* path, int n_layers, int d_sae, s3_compact_host_layer* h_layers)
{
    S3_REQUIRE(path && h_layers, S3_ERR_INVALID_ARG, "null argument");
    File f(fopen(path, "rb"));
    S3_REQUIRE(f != nullptr, S3_ERR_STATE, "cannot open %s", path);
    FileHeader h;
    LayerRecord recs[S3_MAX_SCORE_LAYERS];
    s3_status st = read_header(f.get(), path, &h, recs, S3_MAX_SCORE_LAYERS);
    if (st != S3_OK) return st;
    S3_REQUIRE(static_cast<int>(h.n_layers) == n_layers && static_cast<int>(h.d_sae) == d_sae, S3_ERR_INVALID_ARG,
               "%s holds %u layers of %u features, the caller expects %d of %d", path, h.n_layers, h.d_sae, n_layers, d_sae);
    for (int l = 0; l < n_layers; ++l) {
        s3_compact_host_layer& L = h_layers[l];
        S3_REQUIRE(L.h_row_ptr && L.h_blk_ptr && L.h_payload && ((L.h_blk_first && L.h_blk_desc) || recs[l].n_blocks == 0),
                   S3_ERR_INVALID_ARG, "layer %d: null array", l);
        S3_REQUIRE(L.n_blocks >= recs[l].n_blocks && L.n_words >= recs[l].n_words, S3_ERR_CAPACITY,
                   "layer %d: buffers hold %llu blocks / %llu words, the file has %llu / %llu", l, (unsigned long long)L.n_blocks,
                   (unsigned long long)L.n_words, (unsigned long long)recs[l].n_blocks, (unsigned long long)recs[l].n_words);
    }
    for (int l = 0; l < n_layers; ++l) {
        s3_compact_host_layer& L = h_layers[l];
        L.n_blocks = recs[l].n_blocks;
        L.n_words = recs[l].n_words;
        const bool ok = get(f.get(), L.h_row_ptr, (static_cast<size_t>(d_sae) + 1) * 8) &&
                        get(f.get(), L.h_blk_ptr, (static_cast<size_t>(d_sae) + 1) * 4) && get(f.get(), L.h_blk_first, L.n_blocks * 4) &&
                        get(f.get(), L.h_blk_desc, L.n_blocks * 8) && get(f.get(), L.h_payload, L.n_words * 4);
        S3_REQUIRE(ok, S3_ERR_INVALID_ARG, "%s: cut short inside layer %d", path, l);
        S3_REQUIRE(layer_checksum(L, d_sae) == recs[l].checksum, S3_ERR_INVALID_ARG, "%s: checksum of layer %d does not match", path, l);
        st = check_layer(L, d_sae, l);
        if (st != S3_OK) return st;
    }
    return S3_OK;
}

}  // extern "C"
