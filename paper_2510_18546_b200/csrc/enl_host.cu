// Host side of the library: the paged per-group KV store, the gather plan and the four C-ABI calls.
// Everything here is integer book-keeping plus launches; all arithmetic of the method runs in kernels.
#include <algorithm>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "../../include/enl.h"
#include "enl_internal.h"

using namespace enl;

namespace {

struct Group {
    std::vector<int32_t> pages;       // shared by all layers: positions 16*i .. 16*i+15 live in pages[i]
    std::vector<int32_t> len;         // per layer, -1 = never stored
    // slow tier (Sec. 3.2): pages in the pinned host pool, and which copy is current
    std::vector<int32_t> host_pages;
    bool resident = true;             // the device pages hold the group
    bool host_current = false;        // the host pages hold what the device pages held when last written back
    uint64_t last_use = 0;            // tick of the last enl_step_prepare that selected the group
};

struct DeviceGuard {
    int prev = -1;
    bool switched = false;
    explicit DeviceGuard(int dev)
    {
        if (dev < 0) return;
        if (cudaGetDevice(&prev) == cudaSuccess && prev != dev) {
            cudaSetDevice(dev);
            switched = true;
        }
    }
    ~DeviceGuard()
    {
        if (switched) cudaSetDevice(prev);
    }
};

using EncodeTiledFn = CUresult (*)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                   const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                   CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                   CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    return fn;
}

// bf16 tensor map with 128-byte swizzle; dims/box innermost first, strides in bytes for dims 1..rank-1.
bool encode_map(CUtensorMap *tm, const void *base, int rank, const cuuint64_t *dims, const cuuint64_t *strides,
                const cuuint32_t *box)
{
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, static_cast<cuuint32_t>(rank), const_cast<void *>(base), dims,
              strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

inline int ceil_div(int a, int b) { return (a + b - 1) / b; }

// Tensor maps of the caller's tensors, kept by (pointer, shape): a planning step calls enl_attend once per layer with
// tensors that come back step after step, and encoding three maps per call is most of the host time of a call whose
// gather plan is reused.
struct MapKey {
    const void *base;
    uint64_t d0, d1, d2;
    uint32_t b0, b1, b2;
    bool operator==(const MapKey &o) const
    {
        return base == o.base && d0 == o.d0 && d1 == o.d1 && d2 == o.d2 && b0 == o.b0 && b1 == o.b1 && b2 == o.b2;
    }
};
struct MapCache {
    static constexpr int kSlots = 256;
    MapKey key[kSlots] = {};
    CUtensorMap map[kSlots];
    bool used[kSlots] = {};
    // 3-D bf16 map [d2][d1][d0] with box {b0, b1, b2}
    bool get(CUtensorMap *out, const void *base, const cuuint64_t *dims, const cuuint64_t *strides, const cuuint32_t *box)
    {
        const MapKey k{base, dims[0], dims[1], dims[2], box[0], box[1], box[2]};
        const size_t h = (reinterpret_cast<uintptr_t>(base) >> 8) * 0x9E3779B97F4A7C15ull >> 56;
        for (int probe = 0; probe < 4; ++probe) {
            const int i = static_cast<int>((h + probe) % kSlots);
            if (used[i] && key[i] == k) { *out = map[i]; return true; }
        }
        if (!encode_map(out, base, 3, dims, strides, box)) return false;
        const int i = static_cast<int>(h % kSlots);
        key[i] = k;
        map[i] = *out;
        used[i] = true;
        return true;
    }
};

}  // namespace

struct enl_cache {
    enl_cache_desc_t d{};
    bool gpu = false;
    int rep = 1;
    int n_sm = 148;                         // multiprocessors of the device (grid sizes, split counts)
    int64_t n_pages = 0;
    size_t layer_bytes = 0;                 // one layer of one pool
    uint8_t *kpool = nullptr, *vpool = nullptr;
    std::vector<int32_t> free_pages;        // stack of free page ids (page 0 is never in it)
    std::vector<Group> groups;
    std::vector<CUtensorMap> tm_k, tm_v;    // per layer
    uint64_t epoch = 0;                     // bumped by every store

    // gather plan: host image (pinned when there is a GPU), device copy, capacities
    int32_t cap_entries = 0, cap_items = 0;
    uint8_t *plan_host = nullptr, *plan_dev = nullptr;
    size_t off_eps = 0, off_items = 0, off_stream = 0, off_meta = 0, off_rowslots = 0, off_rowobj = 0, plan_bytes = 0;
    cudaEvent_t plan_copied = nullptr;
    bool plan_valid = false, plan_on_device = false;
    uint64_t plan_epoch = 0;
    int32_t plan_split_hint = 0;
    bool plan_has_mass = false;
    bool plan_direct = false;               // built for a call that wants mass sums or no output: one split, general kernel
    std::vector<int32_t> key_obj;           // object spans the row -> object map was built from
    bool plan_decode = false;               // the plan is for the one-token decode kernel
    bool plan_pair = false;                 // two splits whose CTAs merge inside the attention kernel (cluster of two)
    bool pairs_ok = false;                  // the device can co-schedule two of the attention kernel's CTAs as a cluster
    std::vector<int32_t> key_sel, key_cu, key_len;   // what the current plan was built from
    int32_t plan_entries = 0, plan_items = 0, plan_splits = 1, plan_batch = 0, plan_max_slots = 0;
    MapCache maps;                          // tensor maps of the caller's q / k_new / v_new
    std::vector<int32_t> seen;              // duplicate detection stamps
    int32_t stamp = 0;

    // slow tier
    bool tier = false;
    int64_t n_host_pages = 0;
    size_t host_layer_bytes = 0;
    uint8_t *host_k = nullptr, *host_v = nullptr;           // pinned, [layer][page][kv head][16][D]
    std::vector<int32_t> free_host_pages;
    int2 *pairs_host = nullptr, *pairs_dev = nullptr;        // page moves of one enqueue (pinned staging + device copy)
    int32_t cap_pairs = 0;
    cudaEvent_t pairs_copied = nullptr;
    uint64_t tick = 0;

    float *scratch = nullptr;
    int32_t *status_dev = nullptr;
    int32_t *counters_dev = nullptr;        // decode: finished splits per (episode, kv head)

    EpInfo *h_eps() { return reinterpret_cast<EpInfo *>(plan_host + off_eps); }
    Item *h_items() { return reinterpret_cast<Item *>(plan_host + off_items); }
    int32_t *h_stream() { return reinterpret_cast<int32_t *>(plan_host + off_stream); }
    int32_t *h_meta() { return reinterpret_cast<int32_t *>(plan_host + off_meta); }
    int32_t *h_rowslots() { return reinterpret_cast<int32_t *>(plan_host + off_rowslots); }
    int32_t *h_rowobj() { return reinterpret_cast<int32_t *>(plan_host + off_rowobj); }
};

namespace {

void destroy(enl_cache *c)
{
    if (!c) return;
    if (c->gpu) {
        DeviceGuard g(c->d.device);
        cudaDeviceSynchronize();
        if (c->kpool) cudaFree(c->kpool);
        if (c->vpool) cudaFree(c->vpool);
        if (c->plan_dev) cudaFree(c->plan_dev);
        if (c->plan_host) cudaFreeHost(c->plan_host);
        if (c->scratch) cudaFree(c->scratch);
        if (c->status_dev) cudaFree(c->status_dev);
        if (c->counters_dev) cudaFree(c->counters_dev);
        if (c->plan_copied) cudaEventDestroy(c->plan_copied);
        if (c->host_k) cudaFreeHost(c->host_k);
        if (c->host_v) cudaFreeHost(c->host_v);
        if (c->pairs_host) cudaFreeHost(c->pairs_host);
        if (c->pairs_dev) cudaFree(c->pairs_dev);
        if (c->pairs_copied) cudaEventDestroy(c->pairs_copied);
    } else {
        delete[] c->plan_host;
        delete[] c->pairs_host;
    }
    delete c;
}

int tokens_per_cta(const enl_cache *c) { return kQTiles * (kTileRows / c->rep); }

}  // namespace

extern "C" const char *enl_strerror(int code)
{
    switch (code) {
        case ENL_OK: return "ok";
        case ENL_E_INVAL: return "invalid argument";
        case ENL_E_NOGROUP: return "group id out of range or group never stored for this layer";
        case ENL_E_NOMEM: return "out of pool pages, plan space or memory";
        case ENL_E_CUDA: return "CUDA error, or GPU operation on a bookkeeping-only cache";
        case ENL_E_TIMEOUT: return "a bounded wait inside a kernel expired";
        case ENL_E_LIMIT: return "size beyond the fixed maxima of the entry point that allocates nothing";
        case ENL_E_EVICTED: return "the group is in the slow tier only; enl_step_prepare loads it";
        case ENL_E_CORRUPT: return "a guard page of the pool has been written";
        default: return "unknown error";
    }
}

extern "C" int enl_cache_create(const enl_cache_desc_t *desc, enl_cache_t **out)
{
    if (!desc || !out) return ENL_E_INVAL;
    *out = nullptr;
    enl_cache_desc_t d = *desc;
    if (d.page_tokens == 0) d.page_tokens = kPageTokens;
    if (d.max_batch == 0) d.max_batch = 64;
    if (d.max_q_tokens == 0) d.max_q_tokens = 16384;
    if (d.scratch_bytes == 0) d.scratch_bytes = 64ll << 20;
    if (d.n_layers <= 0 || d.n_q_heads <= 0 || d.n_kv_heads <= 0 || d.n_q_heads % d.n_kv_heads != 0)
        return ENL_E_INVAL;
    const int rep = d.n_q_heads / d.n_kv_heads;
    if (rep != 1 && rep != 2 && rep != 4 && rep != 8 && rep != 16) return ENL_E_INVAL;
    if (d.head_dim != 64 && d.head_dim != 128) return ENL_E_INVAL;
    if (d.page_tokens != kPageTokens || d.dtype != ENL_BF16) return ENL_E_INVAL;
    if (d.max_groups <= 0 || d.max_tokens <= 0 || d.max_batch < 0 || d.max_q_tokens < 0 || d.scratch_bytes < 0)
        return ENL_E_INVAL;
    if (d.device < 0 && d.device != ENL_DEVICE_NONE) return ENL_E_INVAL;

    enl_cache *c = new (std::nothrow) enl_cache;
    if (!c) return ENL_E_NOMEM;
    c->d = d;
    c->rep = rep;
    c->gpu = d.device >= 0;
    // every group may waste up to one page of padding; page 0 stays the all-zero page, and one guard page that is
    // never handed out either closes the pool (enl_cache_selfcheck)
    c->n_pages = (d.max_tokens + kPageTokens - 1) / kPageTokens + d.max_groups + 2;
    if (c->n_pages * d.n_kv_heads * kPageTokens > 0x7fffffffll) { delete c; return ENL_E_INVAL; }
    c->layer_bytes = static_cast<size_t>(c->n_pages) * d.n_kv_heads * kPageTokens * d.head_dim * 2;
    c->groups.resize(d.max_groups);
    c->seen.assign(d.max_groups, 0);
    c->free_pages.reserve(c->n_pages);
    for (int64_t pg = c->n_pages - 2; pg >= 1; --pg) c->free_pages.push_back(static_cast<int32_t>(pg));

    const int tpc = tokens_per_cta(c);
    c->cap_entries = static_cast<int32_t>(std::min<int64_t>(2 * c->n_pages + kPagesPerTile * (d.max_batch + 1), 0x7ffffff0));
    c->cap_items = std::max(4096, (d.max_q_tokens / tpc + d.max_batch + 1) * d.n_kv_heads);
    auto align256 = [](size_t x) { return (x + 255) & ~static_cast<size_t>(255); };
    c->off_eps = 0;
    c->off_items = align256(c->off_eps + sizeof(EpInfo) * d.max_batch);
    c->off_stream = align256(c->off_items + sizeof(Item) * c->cap_items);
    c->off_meta = align256(c->off_stream + sizeof(int32_t) * c->cap_entries);
    c->off_rowslots = align256(c->off_meta + sizeof(int32_t) * c->cap_entries);
    c->off_rowobj = align256(c->off_rowslots + sizeof(int32_t) * d.max_q_tokens);
    c->plan_bytes = align256(c->off_rowobj + sizeof(int32_t) * d.max_q_tokens);

    if (!c->gpu) {
        c->plan_host = new (std::nothrow) uint8_t[c->plan_bytes];
        if (!c->plan_host) { destroy(c); return ENL_E_NOMEM; }
        *out = c;
        return ENL_OK;
    }

    int n_dev = 0;
    if (cudaGetDeviceCount(&n_dev) != cudaSuccess || d.device >= n_dev) { cudaGetLastError(); delete c; return ENL_E_CUDA; }
    DeviceGuard g(d.device);
    if (!get_encode_fn()) { delete c; return ENL_E_CUDA; }
    if (cudaDeviceGetAttribute(&c->n_sm, cudaDevAttrMultiProcessorCount, d.device) != cudaSuccess || c->n_sm < 1) {
        cudaGetLastError();
        delete c;
        return ENL_E_CUDA;
    }
    const size_t pool_bytes = c->layer_bytes * d.n_layers;
    bool okm = cudaMalloc(&c->kpool, pool_bytes) == cudaSuccess && cudaMalloc(&c->vpool, pool_bytes) == cudaSuccess &&
               cudaMalloc(&c->plan_dev, c->plan_bytes) == cudaSuccess &&
               cudaMallocHost(&c->plan_host, c->plan_bytes) == cudaSuccess &&
               cudaMalloc(&c->scratch, static_cast<size_t>(d.scratch_bytes)) == cudaSuccess &&
               cudaMalloc(&c->status_dev, sizeof(int32_t)) == cudaSuccess &&
               cudaMalloc(&c->counters_dev, sizeof(int32_t) * d.max_batch * d.n_kv_heads) == cudaSuccess;
    if (!okm) { cudaGetLastError(); destroy(c); return ENL_E_NOMEM; }
    bool okc = cudaMemset(c->kpool, 0, pool_bytes) == cudaSuccess && cudaMemset(c->vpool, 0, pool_bytes) == cudaSuccess &&
               cudaMemset(c->status_dev, 0, sizeof(int32_t)) == cudaSuccess &&
               cudaMemset(c->counters_dev, 0, sizeof(int32_t) * d.max_batch * d.n_kv_heads) == cudaSuccess &&
               cudaEventCreateWithFlags(&c->plan_copied, cudaEventDisableTiming) == cudaSuccess &&
               cudaEventRecord(c->plan_copied, 0) == cudaSuccess;
    if (!okc) { cudaGetLastError(); destroy(c); return ENL_E_CUDA; }

    c->tm_k.resize(d.n_layers);
    c->tm_v.resize(d.n_layers);
    const cuuint64_t dims[2] = {static_cast<cuuint64_t>(d.head_dim),
                                static_cast<cuuint64_t>(c->n_pages) * d.n_kv_heads * kPageTokens};
    const cuuint64_t strides[1] = {static_cast<cuuint64_t>(d.head_dim) * 2};
    const cuuint32_t box[2] = {64, kPageTokens};
    for (int l = 0; l < d.n_layers; ++l) {
        if (!encode_map(&c->tm_k[l], c->kpool + c->layer_bytes * l, 2, dims, strides, box) ||
            !encode_map(&c->tm_v[l], c->vpool + c->layer_bytes * l, 2, dims, strides, box)) {
            destroy(c);
            return ENL_E_CUDA;
        }
    }
    if (prepare_attention(d.head_dim) != cudaSuccess || prepare_decode(d.head_dim) != cudaSuccess) { cudaGetLastError(); destroy(c); return ENL_E_CUDA; }
    c->pairs_ok = d.head_dim == 128 && attention_pairs_supported();   // else two splits go through the scratch buffer
    if (cudaDeviceSynchronize() != cudaSuccess) { cudaGetLastError(); destroy(c); return ENL_E_CUDA; }
    *out = c;
    return ENL_OK;
}

extern "C" int enl_cache_free(enl_cache_t *c)
{
    destroy(c);
    return ENL_OK;
}

extern "C" int32_t enl_group_len(const enl_cache_t *c, int32_t group_id, int32_t layer)
{
    if (!c) return ENL_E_INVAL;
    if (group_id < 0 || group_id >= c->d.max_groups) return ENL_E_NOGROUP;
    if (layer < 0 || layer >= c->d.n_layers) return ENL_E_INVAL;
    const Group &g = c->groups[group_id];
    return g.len.empty() ? -1 : g.len[layer];
}

extern "C" int enl_cache_status(enl_cache_t *c)
{
    if (!c) return ENL_E_INVAL;
    if (!c->gpu) return ENL_OK;
    DeviceGuard g(c->d.device);
    if (cudaDeviceSynchronize() != cudaSuccess) { cudaGetLastError(); return ENL_E_CUDA; }
    int32_t st = 0;
    if (cudaMemcpy(&st, c->status_dev, sizeof st, cudaMemcpyDeviceToHost) != cudaSuccess) return ENL_E_CUDA;
    if (st != 0) {
        cudaMemset(c->status_dev, 0, sizeof st);
        // a decode launch that gave up may have left its split counters half counted
        cudaMemset(c->counters_dev, 0, sizeof(int32_t) * c->d.max_batch * c->d.n_kv_heads);
        return ENL_E_TIMEOUT;
    }
    return ENL_OK;
}

extern "C" int enl_cache_selfcheck(enl_cache_t *c)
{
    if (!c) return ENL_E_INVAL;
    if (!c->gpu) return ENL_OK;
    DeviceGuard g(c->d.device);
    if (cudaDeviceSynchronize() != cudaSuccess) { cudaGetLastError(); return ENL_E_CUDA; }
    const size_t page_bytes = static_cast<size_t>(c->d.n_kv_heads) * kPageTokens * c->d.head_dim * 2;
    std::vector<uint64_t> buf(page_bytes / 8);
    for (int l = 0; l < c->d.n_layers; ++l)
        for (int kv = 0; kv < 2; ++kv)
            for (int end = 0; end < 2; ++end) {
                const uint8_t *pool = (kv ? c->vpool : c->kpool) + c->layer_bytes * l;
                const uint8_t *page = pool + (end ? static_cast<size_t>(c->n_pages - 1) * page_bytes : 0);
                if (cudaMemcpy(buf.data(), page, page_bytes, cudaMemcpyDeviceToHost) != cudaSuccess) { cudaGetLastError(); return ENL_E_CUDA; }
                for (uint64_t w : buf)
                    if (w != 0) return ENL_E_CORRUPT;
            }
    return ENL_OK;
}

extern "C" int enl_group_store(enl_cache_t *c, int32_t group_id, int32_t layer, int32_t n_tokens, const void *k_dev,
                               const void *v_dev, int32_t mode, void *cuda_stream)
{
    if (!c) return ENL_E_INVAL;
    if (group_id < 0 || group_id >= c->d.max_groups) return ENL_E_NOGROUP;
    if (layer < 0 || layer >= c->d.n_layers || n_tokens < 0) return ENL_E_INVAL;
    if (mode != ENL_REPLACE && mode != ENL_APPEND) return ENL_E_INVAL;
    if (c->gpu && n_tokens > 0) {
        if (!k_dev || !v_dev) return ENL_E_INVAL;
        if ((reinterpret_cast<uintptr_t>(k_dev) | reinterpret_cast<uintptr_t>(v_dev)) & 15) return ENL_E_INVAL;
    }
    Group &g = c->groups[group_id];
    if (!g.resident) return ENL_E_EVICTED;
    const int32_t old_len = g.len.empty() ? -1 : g.len[layer];
    const int64_t new_len64 = (mode == ENL_APPEND && old_len > 0) ? static_cast<int64_t>(old_len) + n_tokens : n_tokens;
    if (new_len64 > 0x3fffffff) return ENL_E_INVAL;
    const int32_t new_len = static_cast<int32_t>(new_len64);
    const int32_t first_pos = new_len - n_tokens;
    const int need_pages = ceil_div(new_len, kPageTokens);
    const int have = static_cast<int>(g.pages.size());
    if (need_pages > have && static_cast<size_t>(need_pages - have) > c->free_pages.size()) return ENL_E_NOMEM;

    // commit the table change
    if (g.len.empty()) g.len.assign(c->d.n_layers, -1);
    for (int i = have; i < need_pages; ++i) {
        g.pages.push_back(c->free_pages.back());
        c->free_pages.pop_back();
    }
    g.len[layer] = new_len;
    g.host_current = false;                                  // the device copy is newer now
    int keep = 0;
    for (int l = 0; l < c->d.n_layers; ++l) keep = std::max(keep, ceil_div(std::max(g.len[l], 0), kPageTokens));
    while (static_cast<int>(g.pages.size()) > keep) {       // pages no layer needs any more
        c->free_pages.push_back(g.pages.back());
        g.pages.pop_back();
    }
    ++c->epoch;

    if (!c->gpu || n_tokens == 0) return ENL_OK;
    DeviceGuard dg(c->d.device);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const size_t row_bytes = static_cast<size_t>(c->d.n_kv_heads) * c->d.head_dim * 2;
    int pos = first_pos;
    while (pos < new_len) {
        PageRun run;
        run.first_page = pos / kPageTokens;
        const int last_page = std::min((new_len - 1) / kPageTokens, run.first_page + kScatterPages - 1);
        for (int i = run.first_page; i <= last_page; ++i) run.ids[i - run.first_page] = g.pages[i];
        const int end = std::min(new_len, (last_page + 1) * kPageTokens);
        const size_t src_off = static_cast<size_t>(pos - first_pos) * row_bytes;
        const int zero_rows = end == new_len ? (kPageTokens - new_len % kPageTokens) % kPageTokens : 0;
        if (launch_page_scatter(c->kpool + c->layer_bytes * layer, c->vpool + c->layer_bytes * layer,
                                static_cast<const uint8_t *>(k_dev) + src_off,
                                static_cast<const uint8_t *>(v_dev) + src_off, run, pos, end - pos, zero_rows,
                                c->d.n_kv_heads, c->d.head_dim, c->n_sm, st) != cudaSuccess) {
            cudaGetLastError();
            return ENL_E_CUDA;
        }
        pos = end;
    }
    return ENL_OK;
}

extern "C" int enl_group_store_all_layers(enl_cache_t *c, int32_t group_id, int32_t n_tokens, const void *const *k_dev,
                                          const void *const *v_dev, int32_t mode, void *cuda_stream)
{
    if (!c) return ENL_E_INVAL;
    if (group_id < 0 || group_id >= c->d.max_groups) return ENL_E_NOGROUP;
    if (n_tokens < 0) return ENL_E_INVAL;
    if (mode != ENL_REPLACE && mode != ENL_APPEND) return ENL_E_INVAL;
    const int L = c->d.n_layers;
    if (c->gpu && n_tokens > 0) {
        if (!k_dev || !v_dev) return ENL_E_INVAL;
        for (int l = 0; l < L; ++l) {
            if (!k_dev[l] || !v_dev[l]) return ENL_E_INVAL;
            if ((reinterpret_cast<uintptr_t>(k_dev[l]) | reinterpret_cast<uintptr_t>(v_dev[l])) & 15) return ENL_E_INVAL;
        }
    }
    Group &g = c->groups[group_id];
    if (!g.resident) return ENL_E_EVICTED;
    const int32_t old_len = g.len.empty() ? -1 : g.len[0];
    for (int l = 1; l < L && !g.len.empty(); ++l)
        if (g.len[l] != old_len) return ENL_E_INVAL;            // the layers must agree before they move together
    const int64_t new_len64 = (mode == ENL_APPEND && old_len > 0) ? static_cast<int64_t>(old_len) + n_tokens : n_tokens;
    if (new_len64 > 0x3fffffff) return ENL_E_INVAL;
    const int32_t new_len = static_cast<int32_t>(new_len64);
    const int32_t first_pos = new_len - n_tokens;
    const int need_pages = ceil_div(new_len, kPageTokens);
    const int have = static_cast<int>(g.pages.size());
    if (need_pages > have && static_cast<size_t>(need_pages - have) > c->free_pages.size()) return ENL_E_NOMEM;

    // commit the table change
    for (int i = have; i < need_pages; ++i) {
        g.pages.push_back(c->free_pages.back());
        c->free_pages.pop_back();
    }
    g.len.assign(L, new_len);
    g.host_current = false;                                  // the device copy is newer now
    while (static_cast<int>(g.pages.size()) > need_pages) { // pages no layer needs any more
        c->free_pages.push_back(g.pages.back());
        g.pages.pop_back();
    }
    ++c->epoch;

    if (!c->gpu || n_tokens == 0) return ENL_OK;
    DeviceGuard dg(c->d.device);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const size_t row_bytes = static_cast<size_t>(c->d.n_kv_heads) * c->d.head_dim * 2;
    for (int layer0 = 0; layer0 < L; layer0 += kScatterLayers) {
        const int nl = std::min(kScatterLayers, L - layer0);
        LayerSrc src;
        for (int l = 0; l < kScatterLayers; ++l) {
            src.k[l] = l < nl ? k_dev[layer0 + l] : nullptr;
            src.v[l] = l < nl ? v_dev[layer0 + l] : nullptr;
        }
        int pos = first_pos;
        while (pos < new_len) {
            PageRun run;
            run.first_page = pos / kPageTokens;
            const int last_page = std::min((new_len - 1) / kPageTokens, run.first_page + kScatterPages - 1);
            for (int i = run.first_page; i <= last_page; ++i) run.ids[i - run.first_page] = g.pages[i];
            const int end = std::min(new_len, (last_page + 1) * kPageTokens);
            const size_t src_off = static_cast<size_t>(pos - first_pos) * row_bytes;
            const int zero_rows = end == new_len ? (kPageTokens - new_len % kPageTokens) % kPageTokens : 0;
            if (launch_page_scatter_layers(c->kpool, c->vpool, c->layer_bytes, layer0, nl, src, src_off, run, pos,
                                           end - pos, zero_rows, c->d.n_kv_heads, c->d.head_dim, c->n_sm, st) != cudaSuccess) {
                cudaGetLastError();
                return ENL_E_CUDA;
            }
            pos = end;
        }
    }
    return ENL_OK;
}

extern "C" int enl_attend(enl_cache_t *c, const enl_attend_args_t *a, void *cuda_stream)
{
    if (!c || !a) return ENL_E_INVAL;
    const enl_cache_desc_t &d = c->d;
    const bool plan_only = (a->flags & ENL_PLAN_ONLY) != 0;
    const bool mass_only = (a->flags & ENL_MASS_ONLY) != 0;
    if (a->flags & ~static_cast<uint32_t>(ENL_PLAN_ONLY | ENL_MASS_ONLY)) return ENL_E_INVAL;
    if (mass_only && !a->group_mass) return ENL_E_INVAL;
    if (!c->gpu && !plan_only) return ENL_E_CUDA;
    if (a->layer < 0 || a->layer >= d.n_layers) return ENL_E_INVAL;
    if (a->batch < 1 || a->batch > d.max_batch) return ENL_E_INVAL;
    if (a->n_sel < 0 || a->n_q < 1 || a->n_new < a->n_q || a->n_q > d.max_q_tokens) return ENL_E_INVAL;
    if (a->n_sel > 0 && !a->sel_ids) return ENL_E_INVAL;
    if (a->split_hint < 0) return ENL_E_INVAL;
    const int B = a->batch;
    if (B > 1 && (!a->cu_sel || !a->cu_q || !a->cu_new)) return ENL_E_INVAL;
    const int32_t one_sel[2] = {0, a->n_sel}, one_q[2] = {0, a->n_q}, one_new[2] = {0, a->n_new};
    const int32_t *cu_sel = a->cu_sel ? a->cu_sel : one_sel;
    const int32_t *cu_q = a->cu_q ? a->cu_q : one_q;
    const int32_t *cu_new = a->cu_new ? a->cu_new : one_new;
    if (cu_sel[0] != 0 || cu_q[0] != 0 || cu_new[0] != 0) return ENL_E_INVAL;
    if (cu_sel[B] != a->n_sel || cu_q[B] != a->n_q || cu_new[B] != a->n_new) return ENL_E_INVAL;
    int max_slots = 0;
    for (int b = 0; b < B; ++b) {
        const int ns = cu_sel[b + 1] - cu_sel[b], nq = cu_q[b + 1] - cu_q[b], nn = cu_new[b + 1] - cu_new[b];
        if (ns < 0 || nq < 1 || nn < nq) return ENL_E_INVAL;
        max_slots = std::max(max_slots, ns);
    }
    if (!plan_only) {
        if (!a->q || !a->k_new || !a->v_new || (!a->out && !mass_only)) return ENL_E_INVAL;
        const uintptr_t al = reinterpret_cast<uintptr_t>(a->q) | reinterpret_cast<uintptr_t>(a->k_new) |
                             reinterpret_cast<uintptr_t>(a->v_new) | reinterpret_cast<uintptr_t>(a->out);
        if (al & 15) return ENL_E_INVAL;
        if (a->group_mass && (reinterpret_cast<uintptr_t>(a->group_mass) & 3)) return ENL_E_INVAL;
    }
    if (a->group_mass && a->mass_stride < max_slots + 1) return ENL_E_INVAL;
    const bool has_sum = a->group_mass_sum != nullptr;
    if (has_sum) {
        if (!a->group_mass || !a->obj_off || a->n_obj < 1 || a->sum_stride < max_slots + 1) return ENL_E_INVAL;
        if (reinterpret_cast<uintptr_t>(a->group_mass_sum) & 3) return ENL_E_INVAL;
        if (a->obj_off[0] < 0 || a->obj_off[a->n_obj] > a->n_q) return ENL_E_INVAL;
        for (int o = 0; o < a->n_obj; ++o)
            if (a->obj_off[o + 1] < a->obj_off[o]) return ENL_E_INVAL;
    }
    const bool direct = has_sum || mass_only;       // these results leave the attention kernel itself: no KV splits

    // ---- select list: ids, duplicates, lengths (Sec. 3.4: a group is selected at most once) ----
    std::vector<int32_t> sel_len(a->n_sel);
    for (int b = 0; b < B; ++b) {
        if (++c->stamp == 0x7fffffff) { std::fill(c->seen.begin(), c->seen.end(), 0); c->stamp = 1; }
        for (int s = cu_sel[b]; s < cu_sel[b + 1]; ++s) {
            const int32_t gid = a->sel_ids[s];
            if (gid < 0 || gid >= d.max_groups) return ENL_E_NOGROUP;
            const Group &g = c->groups[gid];
            if (g.len.empty() || g.len[a->layer] < 0) return ENL_E_NOGROUP;
            if (!g.resident) return ENL_E_EVICTED;
            if (c->seen[gid] == c->stamp) return ENL_E_INVAL;
            c->seen[gid] = c->stamp;
            sel_len[s] = g.len[a->layer];
        }
    }
    if (a->sel_off_out) {
        int32_t *o = a->sel_off_out;
        for (int b = 0; b < B; ++b) {
            int32_t acc = 0;
            *o++ = 0;
            for (int s = cu_sel[b]; s < cu_sel[b + 1]; ++s) { acc += sel_len[s]; *o++ = acc; }
        }
    }

    // ---- gather plan: reuse when nothing it was built from has changed ----
    std::vector<int32_t> cu_key;
    cu_key.reserve(3 * (B + 1));
    cu_key.insert(cu_key.end(), cu_sel, cu_sel + B + 1);
    cu_key.insert(cu_key.end(), cu_q, cu_q + B + 1);
    cu_key.insert(cu_key.end(), cu_new, cu_new + B + 1);
    const bool has_mass = a->group_mass != nullptr;
    bool same_obj = !has_sum;
    if (has_sum)
        same_obj = c->key_obj.size() == static_cast<size_t>(a->n_obj) + 1 &&
                   std::memcmp(c->key_obj.data(), a->obj_off, sizeof(int32_t) * (a->n_obj + 1)) == 0;
    const bool reuse = c->plan_valid && c->plan_epoch == c->epoch && c->plan_split_hint == a->split_hint &&
                       c->plan_has_mass == has_mass && c->plan_direct == direct && same_obj &&
                       c->key_cu == cu_key && c->key_len == sel_len &&
                       c->key_sel.size() == static_cast<size_t>(a->n_sel) &&
                       (a->n_sel == 0 || std::memcmp(c->key_sel.data(), a->sel_ids, sizeof(int32_t) * a->n_sel) == 0);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    DeviceGuard dg(c->gpu ? d.device : -1);

    if (!reuse) {
        // size check first, so that a failed call leaves the previous plan intact
        const int tpc = tokens_per_cta(c);
        int64_t n_entries = 0, base_items = 0;
        int min_tiles = 0x7fffffff;
        for (int b = 0; b < B; ++b) {
            int64_t e = 0;
            for (int s = cu_sel[b]; s < cu_sel[b + 1]; ++s) e += std::max(1, ceil_div(sel_len[s], kPageTokens));
            e = (e + kPagesPerTile - 1) / kPagesPerTile * kPagesPerTile;
            n_entries += e;
            const int nq = cu_q[b + 1] - cu_q[b], nn = cu_new[b + 1] - cu_new[b];
            base_items += static_cast<int64_t>(ceil_div(nq, tpc)) * d.n_kv_heads;
            // fewest tiles any CTA of this episode walks: its first token block
            const int c_first = nn - nq + std::min(tpc, nq) - 1;
            min_tiles = std::min<int64_t>(min_tiles, e / kPagesPerTile + c_first / kTileKeys + 1);
        }
        if (n_entries > c->cap_entries || base_items > c->cap_items) return ENL_E_NOMEM;

        const int slot_stride = max_slots + 1;
        const int64_t per_rh = d.head_dim + 1 + (has_mass ? slot_stride : 0);      // scratch floats per (split, row, head)
        auto fits = [&](int ns) {      // partial O, log-sum-exp and slot log-sums, plus the decode kernel's slot ranges
            return static_cast<int64_t>(ns) * a->n_q * d.n_q_heads * per_rh * 4 +
                   static_cast<int64_t>(ns) * B * d.n_kv_heads * 8 + 16 <= d.scratch_bytes;
        };
        // One query token per episode: the streaming decode kernel, whose CTAs cover at most kDecodeMaxPages
        // pages each and always hand their partial results to the merge kernel.
        bool decode = c->rep <= 8 && !direct;
        int need = 1, fewest = 0x7fffffff;
        for (int b = 0; b < B && decode; ++b) {
            if (cu_q[b + 1] - cu_q[b] != 1) decode = false;
            int64_t e = 0;
            for (int s = cu_sel[b]; s < cu_sel[b + 1]; ++s) e += std::max(1, ceil_div(sel_len[s], kPageTokens));
            e = (e + kPagesPerTile - 1) / kPagesPerTile * kPagesPerTile + ceil_div(cu_new[b + 1] - cu_new[b], kPageTokens);
            need = std::max<int64_t>(need, (e + kDecodeMaxPages - 1) / kDecodeMaxPages);
            fewest = std::min<int64_t>(fewest, e);
        }
        int n_splits = 1;
        if (decode) {
            const int slots = c->n_sm;                                            // one CTA per SM, one wave
            n_splits = a->split_hint >= 1 ? a->split_hint : std::max(1, slots / (B * d.n_kv_heads));
            n_splits = std::min(std::min(std::max(n_splits, need), fewest), kMaxSplits);
            while (n_splits > need && !fits(n_splits)) --n_splits;
            if (n_splits < need || !fits(n_splits) ||
                static_cast<int64_t>(B) * d.n_kv_heads * n_splits > c->cap_items)
                decode = false;                                                    // too long for one merge: general kernel
        }
        if (!decode) {
            n_splits = 1;
            if (direct) n_splits = 1;
            else if (a->split_hint >= 1) n_splits = std::min(a->split_hint, std::max(1, min_tiles));   // no CTA without a tile
            else if (base_items * 5 < c->n_sm * 4) n_splits = std::max(1, std::min(static_cast<int>(c->n_sm / base_items), min_tiles / 2));
            n_splits = std::min<int64_t>(n_splits, std::max<int64_t>(1, c->cap_items / base_items));
            n_splits = std::min(n_splits, kMaxSplits);
            while (n_splits > 1 && !fits(n_splits)) --n_splits;
        }

        if (c->gpu && cudaEventSynchronize(c->plan_copied) != cudaSuccess) { cudaGetLastError(); return ENL_E_CUDA; }
        c->plan_valid = false;
        EpInfo *eps = c->h_eps();
        int32_t *stream = c->h_stream();
        int32_t *smeta = c->h_meta();
        int32_t *rowslots = c->h_rowslots();
        int32_t ne = 0;
        for (int b = 0; b < B; ++b) {
            EpInfo &e = eps[b];
            e.stream_off = ne;
            e.n_slots = cu_sel[b + 1] - cu_sel[b];
            e.q_off = cu_q[b];
            e.n_q = cu_q[b + 1] - cu_q[b];
            e.new_off = cu_new[b];
            e.n_new = cu_new[b + 1] - cu_new[b];
            e.pad = 0;
            for (int s = cu_sel[b]; s < cu_sel[b + 1]; ++s) {
                const int slot = s - cu_sel[b];
                const Group &g = c->groups[a->sel_ids[s]];
                const int len = sel_len[s], np = ceil_div(len, kPageTokens);
                if (np == 0) { stream[ne] = kZeroPage; smeta[ne++] = slot << 8; }
                for (int i = 0; i < np; ++i) {
                    const int nv = std::min(kPageTokens, len - i * kPageTokens);
                    stream[ne] = g.pages[i];
                    smeta[ne++] = (slot << 8) | nv;
                }
            }
            while ((ne - e.stream_off) % kPagesPerTile) { stream[ne] = kZeroPage; smeta[ne++] = (e.n_slots - 1) << 8; }
            e.n_ctiles = (ne - e.stream_off) / kPagesPerTile;
            for (int r = e.q_off; r < e.q_off + e.n_q; ++r) rowslots[r] = e.n_slots;
        }
        if (has_sum) {
            int32_t *rowobj = c->h_rowobj();
            std::fill(rowobj, rowobj + a->n_q, -1);
            for (int o = 0; o < a->n_obj; ++o)
                for (int r = a->obj_off[o]; r < a->obj_off[o + 1]; ++r) rowobj[r] = o;
            c->key_obj.assign(a->obj_off, a->obj_off + a->n_obj + 1);
        } else {
            c->key_obj.clear();
        }
        // CTAs, heaviest first (late token blocks see more new-token tiles)
        struct Work { Item it; int tiles; };
        std::vector<Work> work;
        work.reserve(static_cast<size_t>(base_items) * n_splits);
        for (int b = 0; b < B && decode; ++b)
            for (int h = 0; h < d.n_kv_heads; ++h)
                for (int sp = 0; sp < n_splits; ++sp) work.push_back({Item{b, h, 0, sp}, eps[b].n_ctiles});
        for (int b = 0; b < B && !decode; ++b) {
            const EpInfo &e = eps[b];
            for (int t0 = 0; t0 < e.n_q; t0 += tpc) {
                const int t_hi = std::min(t0 + tpc, e.n_q);
                const int tiles = e.n_ctiles + (e.n_new - e.n_q + t_hi - 1) / kTileKeys + 1;
                for (int h = 0; h < d.n_kv_heads; ++h)
                    for (int sp = 0; sp < n_splits; ++sp) work.push_back({Item{b, h, t0, sp}, tiles});
            }
        }
        std::stable_sort(work.begin(), work.end(), [](const Work &x, const Work &y) { return x.tiles > y.tiles; });
        Item *items = c->h_items();
        for (size_t i = 0; i < work.size(); ++i) items[i] = work[i].it;

        c->plan_entries = ne;
        c->plan_items = static_cast<int32_t>(work.size());
        c->plan_splits = n_splits;
        c->plan_batch = B;
        c->plan_max_slots = max_slots;
        c->plan_epoch = c->epoch;
        c->plan_split_hint = a->split_hint;
        c->plan_has_mass = has_mass;
        c->plan_direct = direct;
        c->plan_decode = decode;
        // Two splits of a head_dim-128 call are launched as clusters of two CTAs, which exchange their partial
        // results through distributed shared memory: no scratch round trip and no merge kernel.  Every CTA must
        // have at least one tile, and the items of a pair must be neighbours (they are: same tile count, stable sort).
        c->plan_pair = !decode && n_splits == 2 && d.head_dim == 128 && min_tiles >= 2 && (c->pairs_ok || !c->gpu);
        c->key_sel.assign(a->sel_ids, a->sel_ids + a->n_sel);
        c->key_cu = cu_key;
        c->key_len = sel_len;
        c->plan_valid = true;
        c->plan_on_device = false;
    }
    if (plan_only) return ENL_OK;

    if (!c->plan_on_device) {
        // one copy covers episodes, items, stream and row->slots (unused gaps travel too; they are small)
        const size_t ent_bytes = sizeof(int32_t) * c->plan_entries;
        bool okc = cudaMemcpyAsync(c->plan_dev, c->plan_host, c->off_stream, cudaMemcpyHostToDevice, st) == cudaSuccess &&
                   (ent_bytes == 0 ||
                    (cudaMemcpyAsync(c->plan_dev + c->off_stream, c->plan_host + c->off_stream, ent_bytes,
                                     cudaMemcpyHostToDevice, st) == cudaSuccess &&
                     cudaMemcpyAsync(c->plan_dev + c->off_meta, c->plan_host + c->off_meta, ent_bytes,
                                     cudaMemcpyHostToDevice, st) == cudaSuccess)) &&
                   cudaMemcpyAsync(c->plan_dev + c->off_rowslots, c->plan_host + c->off_rowslots,
                                   sizeof(int32_t) * a->n_q, cudaMemcpyHostToDevice, st) == cudaSuccess &&
                   (!has_sum || cudaMemcpyAsync(c->plan_dev + c->off_rowobj, c->plan_host + c->off_rowobj,
                                                sizeof(int32_t) * a->n_q, cudaMemcpyHostToDevice, st) == cudaSuccess) &&
                   cudaEventRecord(c->plan_copied, st) == cudaSuccess;
        if (!okc) { cudaGetLastError(); c->plan_valid = false; return ENL_E_CUDA; }
        c->plan_on_device = true;
    }

    const int slot_stride = c->plan_max_slots + 1;
    if (c->plan_decode) {
        DecodeParams dp;
        std::memset(&dp, 0, sizeof dp);
        const cuuint64_t nd[3] = {static_cast<cuuint64_t>(d.head_dim), static_cast<cuuint64_t>(d.n_kv_heads),
                                  static_cast<cuuint64_t>(a->n_new)};
        const cuuint64_t ns[2] = {static_cast<cuuint64_t>(d.head_dim) * 2,
                                  static_cast<cuuint64_t>(d.head_dim) * 2 * d.n_kv_heads};
        const cuuint32_t nb[3] = {64, 1, kPageTokens};
        if (!c->maps.get(&dp.tm_knew, a->k_new, nd, ns, nb) || !c->maps.get(&dp.tm_vnew, a->v_new, nd, ns, nb))
            return ENL_E_CUDA;
        dp.tm_kpool = c->tm_k[a->layer];
        dp.tm_vpool = c->tm_v[a->layer];
        dp.ep0 = c->h_eps()[0];
        dp.eps = reinterpret_cast<const EpInfo *>(c->plan_dev + c->off_eps);
        dp.stream_page = reinterpret_cast<const int32_t *>(c->plan_dev + c->off_stream);
        dp.stream_meta = reinterpret_cast<const int32_t *>(c->plan_dev + c->off_meta);
        dp.q = a->q;
        dp.out = a->out;
        dp.mass = a->group_mass;
        const size_t rows = static_cast<size_t>(c->plan_splits) * a->n_q * d.n_q_heads;
        dp.part_o = c->scratch;
        dp.part_lse = c->scratch + rows * d.head_dim;
        dp.part_slot = has_mass ? c->scratch + rows * (d.head_dim + 1) : nullptr;
        {
            const size_t used = rows * (d.head_dim + 1 + (has_mass ? slot_stride : 0));      // floats
            dp.part_rng = reinterpret_cast<int2 *>(c->scratch + ((used + 1) & ~static_cast<size_t>(1)));
        }
        dp.counters = c->counters_dev;
        dp.status = c->status_dev;
        dp.n_q_total = a->n_q;
        dp.Hq = d.n_q_heads;
        dp.Hkv = d.n_kv_heads;
        dp.rep = c->rep;
        dp.slot_stride = slot_stride;
        dp.mass_stride = a->mass_stride;
        dp.n_splits = c->plan_splits;
        dp.scale_log2 = 1.4426950408889634f / sqrtf(static_cast<float>(d.head_dim));
        if (launch_decode(dp, d.head_dim, c->plan_batch, st) != cudaSuccess) { cudaGetLastError(); return ENL_E_CUDA; }
        return ENL_OK;
    }

    AttnParams p;
    std::memset(&p, 0, sizeof p);
    {
        const cuuint64_t qd[3] = {static_cast<cuuint64_t>(d.head_dim), static_cast<cuuint64_t>(d.n_q_heads),
                                  static_cast<cuuint64_t>(a->n_q)};
        const cuuint64_t qs[2] = {static_cast<cuuint64_t>(d.head_dim) * 2,
                                  static_cast<cuuint64_t>(d.head_dim) * 2 * d.n_q_heads};
        const cuuint32_t qb[3] = {64, static_cast<cuuint32_t>(c->rep), static_cast<cuuint32_t>(kTileRows / c->rep)};
        const cuuint64_t nd[3] = {static_cast<cuuint64_t>(d.head_dim), static_cast<cuuint64_t>(d.n_kv_heads),
                                  static_cast<cuuint64_t>(a->n_new)};
        const cuuint64_t ns[2] = {static_cast<cuuint64_t>(d.head_dim) * 2,
                                  static_cast<cuuint64_t>(d.head_dim) * 2 * d.n_kv_heads};
        const cuuint32_t nb[3] = {64, 1, kTileKeys};
        if (!c->maps.get(&p.tm_q, a->q, qd, qs, qb) || !c->maps.get(&p.tm_knew, a->k_new, nd, ns, nb) ||
            !c->maps.get(&p.tm_vnew, a->v_new, nd, ns, nb))
            return ENL_E_CUDA;
    }
    p.tm_kpool = c->tm_k[a->layer];
    p.tm_vpool = c->tm_v[a->layer];
    p.items = reinterpret_cast<const Item *>(c->plan_dev + c->off_items);
    p.eps = reinterpret_cast<const EpInfo *>(c->plan_dev + c->off_eps);
    p.stream_page = reinterpret_cast<const int32_t *>(c->plan_dev + c->off_stream);
    p.stream_meta = reinterpret_cast<const int32_t *>(c->plan_dev + c->off_meta);
    p.out = a->out;
    p.mass = a->group_mass;
    p.status = c->status_dev;
    p.n_q_total = a->n_q;
    p.Hq = d.n_q_heads;
    p.Hkv = d.n_kv_heads;
    p.rep = c->rep;
    p.mass_stride = a->mass_stride;
    p.n_splits = c->plan_splits;
    p.pair_merge = c->plan_pair ? 1 : 0;
    p.scale_log2 = 1.4426950408889634f / sqrtf(static_cast<float>(d.head_dim));
    p.mass_sum = a->group_mass_sum;
    p.row_obj = has_sum ? reinterpret_cast<const int32_t *>(c->plan_dev + c->off_rowobj) : nullptr;
    p.sum_stride = a->sum_stride;
    p.mass_only = mass_only ? 1 : 0;
    p.first_wave = c->n_sm;
    const bool scratch_merge = p.n_splits > 1 && !c->plan_pair;
    if (scratch_merge) {
        const size_t rows = static_cast<size_t>(p.n_splits) * a->n_q * d.n_q_heads;
        p.part_o = c->scratch;
        p.part_lse = c->scratch + rows * d.head_dim;
        p.part_slot = has_mass ? c->scratch + rows * (d.head_dim + 1) : nullptr;
        p.mass_stride = slot_stride;                 // the partial slot buffer is packed
    }
    if (launch_attention(p, d.head_dim, c->plan_items, st) != cudaSuccess) { cudaGetLastError(); return ENL_E_CUDA; }
    if (scratch_merge) {
        CombineParams cp;
        cp.part_o = p.part_o;
        cp.part_lse = p.part_lse;
        cp.part_slot = p.part_slot;
        cp.out = a->out;
        cp.mass = a->group_mass;
        cp.row_slots = reinterpret_cast<const int32_t *>(c->plan_dev + c->off_rowslots);
        cp.n_q_total = a->n_q;
        cp.Hq = d.n_q_heads;
        cp.D = d.head_dim;
        cp.slot_stride = slot_stride;
        cp.mass_stride = a->mass_stride;
        cp.n_splits = p.n_splits;
        if (launch_combine(cp, st) != cudaSuccess) { cudaGetLastError(); return ENL_E_CUDA; }
    }
    return ENL_OK;
}


// ---- slow tier (Sec. 3.2) -------------------------------------------------------------------------

namespace {

int page_bytes_of(const enl_cache *c) { return c->d.n_kv_heads * kPageTokens * c->d.head_dim * 2; }

// Enqueues the page moves collected in c->pairs_host[0 .. n): direction to_host or to_device.
int enqueue_moves(enl_cache *c, int n, bool to_host, cudaStream_t st)
{
    if (!c->gpu || n == 0) return ENL_OK;
    // the pinned staging list is free again as soon as this upload has run (the event), the device list when the
    // copy kernel behind it has (stream order)
    if (cudaMemcpyAsync(c->pairs_dev, c->pairs_host, sizeof(int2) * n, cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaEventRecord(c->pairs_copied, st) != cudaSuccess) {
        cudaGetLastError();
        return ENL_E_CUDA;
    }
    const cudaError_t e = to_host
        ? launch_page_copy(c->kpool, c->vpool, c->host_k, c->host_v, c->layer_bytes, c->host_layer_bytes, c->pairs_dev, n,
                           c->d.n_layers, page_bytes_of(c), st)
        : launch_page_copy(c->host_k, c->host_v, c->kpool, c->vpool, c->host_layer_bytes, c->layer_bytes, c->pairs_dev, n,
                           c->d.n_layers, page_bytes_of(c), st);
    if (e != cudaSuccess) { cudaGetLastError(); return ENL_E_CUDA; }
    return ENL_OK;
}

// The staging list is reused by the next enqueue: wait until the previous upload of it has been consumed.
bool staging_free(enl_cache *c)
{
    return !c->gpu || cudaEventSynchronize(c->pairs_copied) == cudaSuccess;
}

}  // namespace

extern "C" int enl_tier_enable(enl_cache_t *c, int64_t host_tokens)
{
    if (!c || host_tokens <= 0 || c->tier) return ENL_E_INVAL;
    const int64_t n_host = (host_tokens + kPageTokens - 1) / kPageTokens + c->d.max_groups;
    if (n_host > 0x7fffffffll) return ENL_E_INVAL;
    c->n_host_pages = n_host;
    c->host_layer_bytes = static_cast<size_t>(n_host) * page_bytes_of(c);
    c->cap_pairs = static_cast<int32_t>(std::max<int64_t>(c->n_pages, 16));
    if (c->gpu) {
        DeviceGuard g(c->d.device);
        const size_t bytes = c->host_layer_bytes * c->d.n_layers;
        const bool okm = cudaMallocHost(&c->host_k, bytes) == cudaSuccess && cudaMallocHost(&c->host_v, bytes) == cudaSuccess &&
                         cudaMallocHost(&c->pairs_host, sizeof(int2) * c->cap_pairs) == cudaSuccess &&
                         cudaMalloc(&c->pairs_dev, sizeof(int2) * c->cap_pairs) == cudaSuccess &&
                         cudaEventCreateWithFlags(&c->pairs_copied, cudaEventDisableTiming) == cudaSuccess &&
                         cudaEventRecord(c->pairs_copied, 0) == cudaSuccess;
        if (!okm) {
            cudaGetLastError();
            if (c->host_k) cudaFreeHost(c->host_k);
            if (c->host_v) cudaFreeHost(c->host_v);
            if (c->pairs_host) cudaFreeHost(c->pairs_host);
            if (c->pairs_dev) cudaFree(c->pairs_dev);
            if (c->pairs_copied) cudaEventDestroy(c->pairs_copied);
            c->host_k = c->host_v = nullptr;
            c->pairs_host = c->pairs_dev = nullptr;
            c->pairs_copied = nullptr;
            return ENL_E_NOMEM;
        }
    } else {
        c->pairs_host = new (std::nothrow) int2[c->cap_pairs];
        if (!c->pairs_host) return ENL_E_NOMEM;
    }
    c->free_host_pages.reserve(n_host);
    for (int64_t pg = n_host - 1; pg >= 0; --pg) c->free_host_pages.push_back(static_cast<int32_t>(pg));
    c->tier = true;
    return ENL_OK;
}

extern "C" int enl_group_resident(const enl_cache_t *c, int32_t group_id)
{
    if (!c) return ENL_E_INVAL;
    if (group_id < 0 || group_id >= c->d.max_groups) return ENL_E_NOGROUP;
    return c->groups[group_id].resident ? 1 : 0;
}

namespace {

// Writes group g back (if its host copy is stale) and releases its device pages.  `n` = moves already
// collected in the staging list; returns the new count, or a negative error with nothing changed.
int evict_one(enl_cache *c, Group &g, int n, int64_t *bytes_d2h)
{
    const int np = static_cast<int>(g.pages.size());
    if (!g.host_current) {
        const int have = static_cast<int>(g.host_pages.size());
        if (np > have && static_cast<size_t>(np - have) > c->free_host_pages.size()) return ENL_E_NOMEM;
        if (n + np > c->cap_pairs) return ENL_E_NOMEM;
        for (int i = have; i < np; ++i) { g.host_pages.push_back(c->free_host_pages.back()); c->free_host_pages.pop_back(); }
        while (static_cast<int>(g.host_pages.size()) > np) { c->free_host_pages.push_back(g.host_pages.back()); g.host_pages.pop_back(); }
        for (int i = 0; i < np; ++i) c->pairs_host[n++] = make_int2(g.pages[i], g.host_pages[i]);
        *bytes_d2h += static_cast<int64_t>(np) * page_bytes_of(c) * 2 * c->d.n_layers;
        g.host_current = true;
    }
    for (int i = np - 1; i >= 0; --i) c->free_pages.push_back(g.pages[i]);
    g.pages.clear();
    g.resident = false;
    return n;
}

}  // namespace

extern "C" int enl_group_evict(enl_cache_t *c, int32_t group_id, void *cuda_stream)
{
    if (!c || !c->tier) return ENL_E_INVAL;
    if (group_id < 0 || group_id >= c->d.max_groups) return ENL_E_NOGROUP;
    Group &g = c->groups[group_id];
    if (g.len.empty()) return ENL_E_NOGROUP;
    if (!g.resident) return ENL_OK;
    DeviceGuard dg(c->gpu ? c->d.device : -1);
    if (!staging_free(c)) { cudaGetLastError(); return ENL_E_CUDA; }
    int64_t d2h = 0;
    const int n = evict_one(c, g, 0, &d2h);
    if (n < 0) return n;
    ++c->epoch;
    return enqueue_moves(c, n, true, static_cast<cudaStream_t>(cuda_stream));
}

extern "C" int enl_step_prepare(enl_cache_t *c, const int32_t *sel_ids, int32_t n_sel, void *cuda_stream,
                                enl_prepare_stats_t *stats)
{
    if (!c || !c->tier || n_sel < 0 || (n_sel > 0 && !sel_ids)) return ENL_E_INVAL;
    enl_prepare_stats_t stt = {0, 0, 0, 0, 0};
    // validate, count what has to come in
    int64_t need_pages = 0;
    for (int s = 0; s < n_sel; ++s) {
        const int32_t gid = sel_ids[s];
        if (gid < 0 || gid >= c->d.max_groups) return ENL_E_NOGROUP;
        const Group &g = c->groups[gid];
        if (g.len.empty()) return ENL_E_NOGROUP;
    }
    ++c->tick;
    if (++c->stamp == 0x7fffffff) { std::fill(c->seen.begin(), c->seen.end(), 0); c->stamp = 1; }
    std::vector<int32_t> misses;
    for (int s = 0; s < n_sel; ++s) {
        const int32_t gid = sel_ids[s];
        if (c->seen[gid] == c->stamp) continue;                       // listed twice (several episodes): once is enough
        c->seen[gid] = c->stamp;
        Group &g = c->groups[gid];
        if (g.resident) { ++stt.n_hit; continue; }
        ++stt.n_miss;
        misses.push_back(gid);
        need_pages += static_cast<int64_t>(g.host_pages.size());
    }
    // room in the device pool: evict the least recently selected groups that this step does not use
    std::vector<int32_t> victims;
    int64_t free_after = static_cast<int64_t>(c->free_pages.size());
    if (free_after < need_pages) {
        std::vector<int32_t> cand;
        for (int32_t gid = 0; gid < c->d.max_groups; ++gid) {
            const Group &g = c->groups[gid];
            if (!g.len.empty() && g.resident && !g.pages.empty() && c->seen[gid] != c->stamp) cand.push_back(gid);
        }
        std::sort(cand.begin(), cand.end(), [&](int32_t x, int32_t y) {
            const Group &gx = c->groups[x], &gy = c->groups[y];
            return gx.last_use != gy.last_use ? gx.last_use < gy.last_use : x < y;
        });
        for (int32_t gid : cand) {
            if (free_after >= need_pages) break;
            victims.push_back(gid);
            free_after += static_cast<int64_t>(c->groups[gid].pages.size());
        }
        if (free_after < need_pages) { --c->tick; return ENL_E_NOMEM; }
    }
    // host pages and staging room for the write-backs, checked before anything changes
    {
        int64_t host_need = 0, moves = 0;
        for (int32_t gid : victims) {
            const Group &g = c->groups[gid];
            if (!g.host_current) {
                host_need += std::max<int64_t>(0, static_cast<int64_t>(g.pages.size()) - static_cast<int64_t>(g.host_pages.size()));
                moves += static_cast<int64_t>(g.pages.size());
            }
        }
        if (host_need > static_cast<int64_t>(c->free_host_pages.size()) || moves > c->cap_pairs || need_pages > c->cap_pairs) {
            --c->tick;
            return ENL_E_NOMEM;
        }
    }
    DeviceGuard dg(c->gpu ? c->d.device : -1);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (!victims.empty() || !misses.empty()) ++c->epoch;
    if (!victims.empty()) {
        if (!staging_free(c)) { cudaGetLastError(); return ENL_E_CUDA; }
        int n = 0;
        for (int32_t gid : victims) {
            n = evict_one(c, c->groups[gid], n, &stt.bytes_d2h);
            if (n < 0) return n;                                       // cannot happen: sizes were checked above
            ++stt.n_evicted;
        }
        const int rc = enqueue_moves(c, n, true, st);
        if (rc != ENL_OK) return rc;
    }
    if (!misses.empty()) {
        if (!staging_free(c)) { cudaGetLastError(); return ENL_E_CUDA; }
        int n = 0;
        for (int32_t gid : misses) {
            Group &g = c->groups[gid];
            const int np = static_cast<int>(g.host_pages.size());
            for (int i = 0; i < np; ++i) {
                g.pages.push_back(c->free_pages.back());
                c->free_pages.pop_back();
                c->pairs_host[n++] = make_int2(g.host_pages[i], g.pages[i]);
            }
            g.resident = true;                                         // host copy stays current until the next store
            stt.bytes_h2d += static_cast<int64_t>(np) * page_bytes_of(c) * 2 * c->d.n_layers;
        }
        const int rc = enqueue_moves(c, n, false, st);
        if (rc != ENL_OK) return rc;
    }
    for (int s = 0; s < n_sel; ++s) c->groups[sel_ids[s]].last_use = c->tick;
    if (stats) *stats = stt;
    return ENL_OK;
}

extern "C" int enl_plan_inspect(const enl_cache_t *cc, int32_t cap_entries, int32_t *stream_pages, int32_t *stream_meta,
                                int32_t *n_entries, int32_t cap_batch, int32_t *ep_stream_off,
                                int32_t *ep_cached_tiles, int32_t *n_splits, int32_t *n_items, int32_t *merge_kind)
{
    enl_cache *c = const_cast<enl_cache *>(cc);
    if (!c || !c->plan_valid) return ENL_E_INVAL;
    if (n_entries) *n_entries = c->plan_entries;
    if (n_splits) *n_splits = c->plan_splits;
    if (n_items) *n_items = c->plan_items;
    if (merge_kind) *merge_kind = c->plan_decode ? 3 : c->plan_pair ? 2 : c->plan_splits > 1 ? 1 : 0;
    const int32_t *s = c->h_stream(), *m = c->h_meta();
    for (int i = 0; i < c->plan_entries && i < cap_entries; ++i) {
        if (stream_pages) stream_pages[i] = s[i];
        if (stream_meta) stream_meta[i] = m[i];
    }
    const EpInfo *e = c->h_eps();
    for (int b = 0; b < c->plan_batch && b < cap_batch; ++b) {
        if (ep_stream_off) ep_stream_off[b] = e[b].stream_off;
        if (ep_cached_tiles) ep_cached_tiles[b] = e[b].n_ctiles;
    }
    return ENL_OK;
}
