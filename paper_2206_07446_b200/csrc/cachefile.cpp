// The on-disk model file: kernel plan, raw weights and cached post-transform weights (what the
// paper's decision stage leaves in storage, its Sections 3 and 3.1.2), and the reader that feeds
// a cold run from it.  Host code only.
//
// Layout, all integers little-endian:
//   header, 64 bytes: magic "NNV12WC\0", u32 version = 1, u32 n_layers, u64 w_bytes, u64 c_bytes,
//       u64 raw_off = round_up(64 + 88 n, 4096), u64 cached_off = raw_off + round_up(w_bytes, 4096),
//       u32 n_little, u32 0, u64 FNV-1a-64 of the two tables
//   layer table: n x nnv_layer_desc_t (14 x i32, 2 x u64 = 72 bytes)
//   plan table:  n x { i32 variant, math, cached, queue }   (-1 -1 0 -1 for pool layers)
//   zero padding, raw blob at raw_off, zero padding, cached blob at cached_off, zero padding to 4096.
#include <errno.h>
#include <fcntl.h>
#include <string.h>
#include <sys/stat.h>
#include <unistd.h>

#include <string>
#include <vector>

#include "nnv_internal.h"

using namespace nnv;

struct nnv_cache {
    int fd = -1;
    std::string path;
    uint32_t n_layers = 0, n_little = 0;
    uint64_t w_bytes = 0, c_bytes = 0, raw_off = 0, cached_off = 0, file_bytes = 0;
    std::vector<nnv_layer_desc_t> layers;
    std::vector<nnv_choice_t> choices;
    std::vector<int32_t> queue_of;
};

namespace {

constexpr uint64_t PAGE = 4096;
constexpr char MAGIC[8] = {'N', 'N', 'V', '1', '2', 'W', 'C', '\0'};
static_assert(sizeof(nnv_layer_desc_t) == 72, "the layer table stores nnv_layer_desc_t as it is");

struct PlanRow { int32_t variant, math, cached, queue; };

#pragma pack(push, 1)
struct FileHeader {
    char magic[8];
    uint32_t version, n_layers;
    uint64_t w_bytes, c_bytes, raw_off, cached_off;
    uint32_t n_little, zero;
    uint64_t table_hash;
};
#pragma pack(pop)
static_assert(sizeof(FileHeader) == 64, "header is 64 bytes");

uint64_t fnv1a64(const uint8_t* p, size_t n) {
    uint64_t h = 0xCBF29CE484222325ull;
    for (size_t i = 0; i < n; ++i) {
        h ^= p[i];
        h *= 0x100000001B3ull;
    }
    return h;
}

nnv_status_t write_all(int fd, const void* buf, uint64_t n, uint64_t off) {
    const uint8_t* p = (const uint8_t*)buf;
    while (n) {
        const ssize_t w = pwrite(fd, p, (size_t)std::min<uint64_t>(n, 1u << 30), (off_t)off);
        if (w < 0 && errno == EINTR) continue;
        NNV_REQUIRE(w > 0, NNV_ERR_STATE, "write failed: %s", strerror(errno));
        p += w; n -= (uint64_t)w; off += (uint64_t)w;
    }
    return NNV_OK;
}

}  // namespace

namespace nnv {

nnv_status_t cache_read_range(const nnv_cache* c, uint64_t off, void* dst, uint64_t n) {
    uint8_t* p = (uint8_t*)dst;
    while (n) {
        const ssize_t r = pread(c->fd, p, (size_t)std::min<uint64_t>(n, 1u << 30), (off_t)off);
        if (r < 0 && errno == EINTR) continue;
        NNV_REQUIRE(r > 0, NNV_ERR_STATE, "read of %s failed at offset %llu: %s", c->path.c_str(), (unsigned long long)off,
                    r == 0 ? "end of file" : strerror(errno));
        p += r; n -= (uint64_t)r; off += (uint64_t)r;
    }
    return NNV_OK;
}

void cache_geometry(const nnv_cache* c, uint64_t* raw_off, uint64_t* cached_off, uint64_t* w_bytes, uint64_t* c_bytes,
                    const nnv_choice_t** file_choices, int* n_layers) {
    *raw_off = c->raw_off; *cached_off = c->cached_off; *w_bytes = c->w_bytes; *c_bytes = c->c_bytes;
    *file_choices = c->choices.data(); *n_layers = (int)c->n_layers;
}

const nnv_layer_desc_t* cache_layers(const nnv_cache* c) { return c->layers.data(); }

}  // namespace nnv

extern "C" {

nnv_status_t nnv_cache_write(const char* path, const nnv_plan_t* p, const nnv_choice_t* choices, const int32_t* queue_of,
                             int32_t n_little, const void* h_weights, uint64_t w_bytes, const void* h_cached,
                             uint64_t c_bytes) {
    NNV_REQUIRE(path && p && choices && h_weights, NNV_ERR_INVALID_ARG, "null argument");
    NNV_REQUIRE(n_little >= 0 && n_little <= NNV_MAX_QUEUES && (queue_of || n_little == 0), NNV_ERR_INVALID_ARG,
                "a schedule needs queue_of and n_little in 1..%d", NNV_MAX_QUEUES);
    const int n = (int)p->layers.size();
    std::vector<uint64_t> coff(n);
    uint64_t ctotal = 0;
    NNV_TRY(nnv_cached_layout(p, choices, coff.data(), &ctotal));
    NNV_REQUIRE(ctotal == 0 || (h_cached && c_bytes >= ctotal), NNV_ERR_INVALID_ARG, "cached blob needs %llu bytes",
                (unsigned long long)ctotal);
    if (!h_cached) c_bytes = 0;
    std::vector<uint8_t> tables((size_t)n * (sizeof(nnv_layer_desc_t) + sizeof(PlanRow)));
    memcpy(tables.data(), p->layers.data(), (size_t)n * sizeof(nnv_layer_desc_t));
    PlanRow* rows = reinterpret_cast<PlanRow*>(tables.data() + (size_t)n * sizeof(nnv_layer_desc_t));
    for (int i = 0; i < n; ++i) {
        if (p->layers[i].op != NNV_OP_CONV) {
            rows[i] = PlanRow{-1, -1, 0, -1};
            continue;
        }
        NNV_TRY(check_choice(*p, i, choices[i].variant, choices[i].math));
        const nnv_layer_desc_t& L = p->layers[i];
        NNV_REQUIRE(L.w_off + raw_weight_bytes(L) <= w_bytes && (!L.has_bias || L.b_off + 4ull * L.K <= w_bytes),
                    NNV_ERR_INVALID_ARG, "layer %d: weights lie outside the weight blob", i);
        NNV_REQUIRE(!queue_of || n_little == 0 || (queue_of[i] >= 0 && queue_of[i] <= n_little), NNV_ERR_INVALID_ARG,
                    "layer %d: queue %d outside 0..%d", i, queue_of ? queue_of[i] : 0, n_little);
        rows[i] = PlanRow{choices[i].variant, choices[i].math, choices[i].cached, (queue_of && n_little) ? queue_of[i] : -1};
    }
    FileHeader h{};
    memcpy(h.magic, MAGIC, 8);
    h.version = 1; h.n_layers = (uint32_t)n;
    h.w_bytes = w_bytes; h.c_bytes = c_bytes;
    h.raw_off = align_up(sizeof(FileHeader) + tables.size(), PAGE);
    h.cached_off = h.raw_off + align_up(w_bytes, PAGE);
    h.n_little = (uint32_t)n_little; h.zero = 0;
    h.table_hash = fnv1a64(tables.data(), tables.size());
    const uint64_t file_bytes = h.cached_off + align_up(c_bytes, PAGE);

    const int fd = open(path, O_WRONLY | O_CREAT | O_TRUNC, 0644);
    NNV_REQUIRE(fd >= 0, NNV_ERR_STATE, "cannot create %s: %s", path, strerror(errno));
    nnv_status_t rc = NNV_OK;
    if (ftruncate(fd, (off_t)file_bytes) != 0) rc = fail(NNV_ERR_STATE, "cannot size %s: %s", path, strerror(errno));   // gaps read as zero
    if (rc == NNV_OK) rc = write_all(fd, &h, sizeof(h), 0);
    if (rc == NNV_OK) rc = write_all(fd, tables.data(), tables.size(), sizeof(h));
    if (rc == NNV_OK) rc = write_all(fd, h_weights, w_bytes, h.raw_off);
    if (rc == NNV_OK && c_bytes) rc = write_all(fd, h_cached, c_bytes, h.cached_off);
    if (rc == NNV_OK && fsync(fd) != 0) rc = fail(NNV_ERR_STATE, "fsync of %s failed: %s", path, strerror(errno));
    close(fd);
    return rc;
}

nnv_status_t nnv_cache_open(const char* path, nnv_cache_t** out) {
    NNV_REQUIRE(path && out, NNV_ERR_INVALID_ARG, "null argument");
    nnv_cache* c = new (std::nothrow) nnv_cache();
    NNV_REQUIRE(c, NNV_ERR_STATE, "out of host memory");
    c->path = path;
    c->fd = open(path, O_RDONLY);
    nnv_status_t rc = NNV_OK;
    auto body = [&]() -> nnv_status_t {
        NNV_REQUIRE(c->fd >= 0, NNV_ERR_STATE, "cannot open %s: %s", path, strerror(errno));
        struct stat st;
        NNV_REQUIRE(fstat(c->fd, &st) == 0, NNV_ERR_STATE, "cannot stat %s: %s", path, strerror(errno));
        c->file_bytes = (uint64_t)st.st_size;
        NNV_REQUIRE(c->file_bytes >= sizeof(FileHeader), NNV_ERR_INVALID_ARG, "%s is shorter than a model-file header", path);
        FileHeader h;
        NNV_TRY(cache_read_range(c, 0, &h, sizeof(h)));
        NNV_REQUIRE(memcmp(h.magic, MAGIC, 8) == 0 && h.version == 1, NNV_ERR_INVALID_ARG, "%s is not a version-1 model file", path);
        NNV_REQUIRE(h.n_layers > 0 && h.n_layers <= 4096, NNV_ERR_INVALID_ARG, "%s: layer count %u out of range", path, h.n_layers);
        const uint64_t tlen = (uint64_t)h.n_layers * (sizeof(nnv_layer_desc_t) + sizeof(PlanRow));
        NNV_REQUIRE(h.raw_off == align_up(sizeof(FileHeader) + tlen, PAGE) && h.cached_off == h.raw_off + align_up(h.w_bytes, PAGE) &&
                        c->file_bytes == h.cached_off + align_up(h.c_bytes, PAGE) && h.n_little <= NNV_MAX_QUEUES,
                    NNV_ERR_INVALID_ARG, "%s: inconsistent offsets or file size", path);
        std::vector<uint8_t> tables((size_t)tlen);
        NNV_TRY(cache_read_range(c, sizeof(FileHeader), tables.data(), tlen));
        NNV_REQUIRE(fnv1a64(tables.data(), tables.size()) == h.table_hash, NNV_ERR_INVALID_ARG, "%s: table hash mismatch", path);
        c->n_layers = h.n_layers; c->n_little = h.n_little;
        c->w_bytes = h.w_bytes; c->c_bytes = h.c_bytes; c->raw_off = h.raw_off; c->cached_off = h.cached_off;
        c->layers.resize(h.n_layers);
        memcpy(c->layers.data(), tables.data(), (size_t)h.n_layers * sizeof(nnv_layer_desc_t));
        const PlanRow* rows = reinterpret_cast<const PlanRow*>(tables.data() + (size_t)h.n_layers * sizeof(nnv_layer_desc_t));
        c->choices.resize(h.n_layers);
        c->queue_of.resize(h.n_layers);
        for (uint32_t i = 0; i < h.n_layers; ++i) {
            c->choices[i] = nnv_choice_t{rows[i].variant, rows[i].math, rows[i].cached};
            c->queue_of[i] = rows[i].queue;
        }
        return NNV_OK;
    };
    rc = body();
    if (rc != NNV_OK) {
        if (c->fd >= 0) close(c->fd);
        delete c;
        return rc;
    }
    *out = c;
    return NNV_OK;
}

nnv_status_t nnv_cache_close(nnv_cache_t* c) {
    if (!c) return NNV_OK;
    if (c->fd >= 0) close(c->fd);
    delete c;
    return NNV_OK;
}

nnv_status_t nnv_cache_info(const nnv_cache_t* c, int32_t* n_layers, uint64_t* w_bytes, uint64_t* c_bytes, int32_t* n_little,
                            uint64_t* file_bytes) {
    NNV_REQUIRE(c, NNV_ERR_INVALID_ARG, "null argument");
    if (n_layers) *n_layers = (int32_t)c->n_layers;
    if (w_bytes) *w_bytes = c->w_bytes;
    if (c_bytes) *c_bytes = c->c_bytes;
    if (n_little) *n_little = (int32_t)c->n_little;
    if (file_bytes) *file_bytes = c->file_bytes;
    return NNV_OK;
}

nnv_status_t nnv_cache_read_plan(const nnv_cache_t* c, nnv_layer_desc_t* layers, nnv_choice_t* choices, int32_t* queue_of,
                                 int32_t cap) {
    NNV_REQUIRE(c && layers && choices, NNV_ERR_INVALID_ARG, "null argument");
    NNV_REQUIRE(cap >= (int32_t)c->n_layers, NNV_ERR_INVALID_ARG, "output capacity %d too small for %u layers", cap, c->n_layers);
    for (uint32_t i = 0; i < c->n_layers; ++i) {
        layers[i] = c->layers[i];
        choices[i] = c->choices[i];
        if (queue_of) queue_of[i] = c->queue_of[i];
    }
    return NNV_OK;
}

nnv_status_t nnv_cache_read_blobs(const nnv_cache_t* c, void* h_weights, uint64_t w_cap, void* h_cached, uint64_t c_cap) {
    NNV_REQUIRE(c && h_weights, NNV_ERR_INVALID_ARG, "null argument");
    NNV_REQUIRE(w_cap >= c->w_bytes && (!h_cached || c_cap >= c->c_bytes), NNV_ERR_WORKSPACE_TOO_SMALL, "buffers too small for the blobs");
    NNV_TRY(cache_read_range(c, c->raw_off, h_weights, c->w_bytes));
    if (h_cached && c->c_bytes) NNV_TRY(cache_read_range(c, c->cached_off, h_cached, c->c_bytes));
    return NNV_OK;
}

nnv_status_t nnv_cache_drop_pages(const nnv_cache_t* c) {
    NNV_REQUIRE(c, NNV_ERR_INVALID_ARG, "null argument");
    const int rc = posix_fadvise(c->fd, 0, 0, POSIX_FADV_DONTNEED);
    NNV_REQUIRE(rc == 0, NNV_ERR_STATE, "posix_fadvise on %s failed: %s", c->path.c_str(), strerror(rc));
    return NNV_OK;
}

}  // extern "C"
