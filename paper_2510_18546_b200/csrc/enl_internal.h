// Internal declarations shared by the host side and the kernels of the library.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace enl {

constexpr int kPageTokens = 16;     // tokens per page: one TMA box of 16 rows x 128 B per 64 channels
constexpr int kTileKeys   = 128;    // keys per KV tile (8 pages)
constexpr int kPagesPerTile = kTileKeys / kPageTokens;
constexpr int kTileRows   = 128;    // query rows per Q tile = (128 / rep) tokens x rep q heads of one kv head
constexpr int kQTiles     = 2;      // Q tiles per CTA (they share every K/V tile the CTA loads)
constexpr int kZeroPage   = 0;      // page 0 is never handed out: all zeros, target of null stream entries

// One episode of an attend call.
struct EpInfo {
    int32_t stream_off;     // first KV-stream entry (multiple of kPagesPerTile)
    int32_t n_ctiles;       // cached tiles (128 keys each, last one padded with null entries)
    int32_t n_slots;        // selected groups G_b; mass slot G_b = new tokens
    int32_t q_off, n_q;     // first query row (global) and count
    int32_t new_off, n_new; // first new-token key (global) and count
    int32_t pad;
};

// One CTA of the attention launch.
struct Item {
    int32_t ep;             // episode
    int32_t kvh;            // kv head
    int32_t t0;             // first query token (episode-relative) of the CTA's two Q tiles
    int32_t split;          // KV split index in [0, n_splits)
};

// Kernel parameters (passed by value as a __grid_constant__).
struct AttnParams {
    CUtensorMap tm_q;       // [n_q][Hq][D]      box {64, rep, 128/rep}
    CUtensorMap tm_knew;    // [n_new][Hkv][D]   box {64, 1, 128}
    CUtensorMap tm_vnew;
    CUtensorMap tm_kpool;   // [pages*Hkv*16][D] box {64, 16}   (one layer)
    CUtensorMap tm_vpool;
    const Item   *items;
    const EpInfo *eps;
    const int32_t *stream_page;   // KV stream: page id of every entry
    const int32_t *stream_meta;   // KV stream: slot << 8 | valid tokens
    void   *out;            // bf16 [n_q][Hq][D]
    float  *mass;           // fp32 or null
    float  *part_o;         // split mode: [split][row][Hq][D] fp32 (normalised by the split's own sum)
    float  *part_lse;       // split mode: [split][row][Hq] log2-sum-exp of the split
    float  *part_slot;      // split mode: [split][row][Hq][mass_stride] per-slot log2-sum-exp
    int32_t *status;        // device word: nonzero = a bounded wait expired
    int32_t n_q_total;      // rows over the batch
    int32_t Hq, Hkv, rep;   // rep = Hq / Hkv
    int32_t mass_stride;
    int32_t n_splits;
    int32_t pair_merge;     // 1: two splits, launched as clusters of two CTAs that merge through distributed shared memory
    float   scale_log2;     // log2(e) / sqrt(D)
    float  *mass_sum;       // fp32 [n_obj][sum_stride] or null: per object the masses summed over its rows and the q heads (added to)
    const int32_t *row_obj; // [n_q_total]: object of every query row, -1 = none (only with mass_sum)
    int32_t sum_stride;
    int32_t mass_only;      // 1: the output rows are not written
    int32_t first_wave;     // CTAs that start while the previous kernel of the stream may still run (the number of SMs)
};

// Decode (one query token per episode): pages of the key stream one CTA may cover, and the most splits
// the merge kernel takes.
constexpr int kDecodeMaxPages = 256;
constexpr int kMaxSplits      = 64;

struct DecodeParams {
    CUtensorMap tm_knew;    // [n_new][Hkv][D]   box {64, 1, 16}
    CUtensorMap tm_vnew;
    CUtensorMap tm_kpool;   // [pages*Hkv*16][D] box {64, 16}   (one layer)
    CUtensorMap tm_vpool;
    EpInfo ep0;             // episode 0 (used when the call has one episode; grid = splits x kv heads x episodes)
    const EpInfo *eps;
    const int32_t *stream_page;
    const int32_t *stream_meta;
    const void *q;          // bf16 [n_q][Hq][D], one row per episode
    void   *out;            // bf16 [n_q][Hq][D]
    float  *mass;           // fp32 or null
    float  *part_o, *part_lse, *part_slot;      // as in AttnParams; part_slot is null when mass is
    int2   *part_rng;       // [split][episode][kv head]: first slot and number of slots the split's range touched
    int32_t *counters;      // [episode][kv head], zero between launches: splits that have finished
    int32_t *status;
    int32_t n_q_total;
    int32_t Hq, Hkv, rep;
    int32_t slot_stride;    // row stride of part_slot
    int32_t mass_stride;    // row stride of mass
    int32_t n_splits;
    float   scale_log2;
};

struct CombineParams {
    const float *part_o, *part_lse, *part_slot;
    void  *out;
    float *mass;
    const int32_t *row_slots;   // [n_q_total]: G_b of the row's episode
    int32_t n_q_total, Hq, D;
    int32_t slot_stride;        // row stride of part_slot
    int32_t mass_stride;        // row stride of mass
    int32_t n_splits;
};

// Programmatic dependent launch: a kernel launched this way may start (set-up only) while the previous kernel
// of the stream is still draining; it must execute pdl_wait() before it touches anything a predecessor may have
// written, and pdl_trigger() as early as it likes so that its own successor can be set up the same way.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
template <typename Kernel, typename Params>
inline cudaError_t launch_pdl(Kernel kernel, dim3 grid, dim3 block, size_t smem, cudaStream_t st, const Params &prm,
                              unsigned cluster_x = 1)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cluster_x > 1) {                                     // grid.x must be a multiple of cluster_x
        attr[1].id = cudaLaunchAttributeClusterDimension;
        attr[1].val.clusterDim.x = cluster_x;
        attr[1].val.clusterDim.y = 1;
        attr[1].val.clusterDim.z = 1;
        cfg.numAttrs = 2;
    }
    return cudaLaunchKernelEx(&cfg, kernel, prm);
}
// the same for kernels that take several plain arguments
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl_n(void (*kernel)(KArgs...), dim3 grid, dim3 block, cudaStream_t st, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif

// launchers (defined in the .cu files of the kernels)
cudaError_t launch_attention(const AttnParams &p, int head_dim, int n_items, cudaStream_t st);
cudaError_t launch_combine(const CombineParams &p, cudaStream_t st);
cudaError_t launch_decode(const DecodeParams &p, int head_dim, int batch, cudaStream_t st);
cudaError_t prepare_decode(int head_dim);
size_t decode_smem_bytes(int head_dim);
// Page ids of (part of) one group, passed by value to the scatter kernel.
constexpr int kScatterPages = 64;
struct PageRun {
    int32_t ids[kScatterPages];   // ids[i] = page holding group positions (first_page + i)*16 ..
    int32_t first_page;           // index within the group of ids[0]
};
// zero_rows: rows behind the last token of the run's last page that are cleared (the group ends there)
cudaError_t launch_page_scatter(void *kpool_layer, void *vpool_layer, const void *k, const void *v,
                                const PageRun &run, int first_pos, int n_tokens, int zero_rows,
                                int Hkv, int D, int n_sm, cudaStream_t st);
// The same for up to kScatterLayers layers in one launch: layer l reads k[l] + src_off, v[l] + src_off (bytes)
// and writes the pool of layer layer0 + l.
constexpr int kScatterLayers = 64;
struct LayerSrc {
    const void *k[kScatterLayers];
    const void *v[kScatterLayers];
};
cudaError_t launch_page_scatter_layers(void *kpool, void *vpool, size_t layer_bytes, int layer0, int n_layers,
                                       const LayerSrc &src, size_t src_off, const PageRun &run, int first_pos,
                                       int n_tokens, int zero_rows, int Hkv, int D, int n_sm, cudaStream_t st);
// Copies whole pages (all kv heads) between two pools of the page format, every layer, K and V: pairs[i] =
// {source page, destination page}; the pools may be device memory or pinned host memory.
cudaError_t launch_page_copy(const uint8_t *src_k, const uint8_t *src_v, uint8_t *dst_k, uint8_t *dst_v,
                             size_t src_layer_bytes, size_t dst_layer_bytes, const int2 *pairs, int n_pairs,
                             int n_layers, int page_bytes, cudaStream_t st);
size_t attention_smem_bytes(int head_dim);
// Opts the attention kernel into its dynamic shared memory size on the current device.
cudaError_t prepare_attention(int head_dim);
// can the device run the head_dim-128 kernel as clusters of two CTAs (the in-kernel merge of two KV splits)?
bool attention_pairs_supported();

}  // namespace enl
