// Small kernels around the attention: scatter of a group's K/V rows into pool pages (the store of
// Sec. 3.2 "Discrete Memory Caching") and the merge of KV splits (log-sum-exp weighted average of the
// partial outputs, sum of the partial per-slot masses).
#include <cuda_bf16.h>

#include <algorithm>

#include "enl_internal.h"

namespace enl {
namespace {

// k, v: [n_tokens][Hkv][D] bf16 -> pool layer [page][Hkv][16][D]; 16-byte chunks, one per thread-iteration.
// The `zero_rows` rows behind the last token (the padding of the group's last page) are cleared: the attention
// kernels give padded keys probability 0, and 0 times whatever an earlier, longer version of the group left
// there must stay 0 (a stale non-finite value would not).
__device__ __forceinline__ void scatter_rows(uint4 *__restrict__ kpool, uint4 *__restrict__ vpool, const uint4 *__restrict__ k,
                                             const uint4 *__restrict__ v, const PageRun &run, int first_pos, int n_tokens,
                                             int zero_rows, int Hkv, int chunks_per_row)
{
    const long long total = static_cast<long long>(n_tokens + zero_rows) * Hkv * chunks_per_row;
    const long long n_src = static_cast<long long>(n_tokens) * Hkv * chunks_per_row;
    for (long long id = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; id < total;
         id += static_cast<long long>(gridDim.x) * blockDim.x) {
        const int ch = static_cast<int>(id % chunks_per_row);
        const long long th = id / chunks_per_row;
        const int head = static_cast<int>(th % Hkv);
        const int tok = static_cast<int>(th / Hkv);
        const int pos = first_pos + tok;
        const int page = run.ids[pos / kPageTokens - run.first_page];
        const long long dst = ((static_cast<long long>(page) * Hkv + head) * kPageTokens + pos % kPageTokens) *
                                  chunks_per_row + ch;
        const bool real = id < n_src;
        kpool[dst] = real ? k[id] : make_uint4(0u, 0u, 0u, 0u);
        vpool[dst] = real ? v[id] : make_uint4(0u, 0u, 0u, 0u);
    }
}
__global__ void page_scatter_kernel(uint4 *__restrict__ kpool, uint4 *__restrict__ vpool,
                                    const uint4 *__restrict__ k, const uint4 *__restrict__ v,
                                    const __grid_constant__ PageRun run, int first_pos, int n_tokens, int zero_rows,
                                    int Hkv, int chunks_per_row)
{
    pdl_trigger();
    pdl_wait();                                             // an attention kernel may still be reading these pages
    scatter_rows(kpool, vpool, k, v, run, first_pos, n_tokens, zero_rows, Hkv, chunks_per_row);
}

// grid (blocks, layers): the same scatter for several layers of one group at once
__global__ void page_scatter_layers_kernel(uint4 *__restrict__ kpool, uint4 *__restrict__ vpool, long long layer_chunks,
                                           const __grid_constant__ LayerSrc src, long long src_chunk_off,
                                           const __grid_constant__ PageRun run, int first_pos, int n_tokens,
                                           int zero_rows, int Hkv, int chunks_per_row)
{
    const uint4 *k = static_cast<const uint4 *>(src.k[blockIdx.y]) + src_chunk_off;
    const uint4 *v = static_cast<const uint4 *>(src.v[blockIdx.y]) + src_chunk_off;
    uint4 *kp = kpool + layer_chunks * blockIdx.y, *vp = vpool + layer_chunks * blockIdx.y;
    pdl_trigger();
    pdl_wait();                                             // an attention kernel may still be reading these pages
    scatter_rows(kp, vp, k, v, run, first_pos, n_tokens, zero_rows, Hkv, chunks_per_row);
}

__device__ __forceinline__ float ex2f(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// One warp per (query row, q head): lane l merges channels 4l..4l+3 (D = 128) or 2l, 2l+1 (D = 64),
// then the lanes stride over the slots.
template <int D>
__global__ void combine_kernel(const CombineParams p)
{
    constexpr int V = D / 32;                               // channels per lane
    const int lane = threadIdx.x & 31;
    const long long rh = blockIdx.x * static_cast<long long>(blockDim.x >> 5) + (threadIdx.x >> 5);
    const long long split_stride = static_cast<long long>(p.n_q_total) * p.Hq;
    pdl_trigger();
    pdl_wait();                                             // the partial results come from the previous kernel
    if (rh >= split_stride) return;
    const int row = static_cast<int>(rh / p.Hq);
    const float ninf = -__builtin_huge_valf();

    // Few splits (the usual case): every load of the warp -- log-sum-exps, partial outputs, the first 32 slot
    // log-sums -- is issued before anything is computed, so the warp pays one memory round trip, not five.
    if (p.n_splits <= 4) {
        const float *slot0 = p.part_slot ? p.part_slot + rh * p.slot_stride + lane : nullptr;
        const int G = p.mass ? p.row_slots[row] : -1;
        float lv[4], sv[4], ov[4][V];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const bool on = k < p.n_splits;
            lv[k] = on ? __ldcg(p.part_lse + k * split_stride + rh) : ninf;
            sv[k] = (on && p.mass && lane <= G) ? __ldcg(slot0 + k * split_stride * p.slot_stride) : ninf;
            const float *src = p.part_o + ((on ? k : 0) * split_stride + rh) * D + lane * V;
            if constexpr (V == 4) {
                const float4 t = __ldcg(reinterpret_cast<const float4 *>(src));
                ov[k][0] = t.x; ov[k][1] = t.y; ov[k][2] = t.z; ov[k][3] = t.w;
            } else {
                const float2 t = __ldcg(reinterpret_cast<const float2 *>(src));
                ov[k][0] = t.x; ov[k][1] = t.y;
            }
        }
        const float mxv = fmaxf(fmaxf(lv[0], lv[1]), fmaxf(lv[2], lv[3]));
        float sum = 0.f;
#pragma unroll
        for (int k = 0; k < 4; ++k) sum += (lv[k] != ninf) ? ex2f(lv[k] - mxv) : 0.f;
        const float lse = mxv + log2f(sum);
        const float lse_s = (lse > ninf) ? lse : 0.f;
        float acc[V];
#pragma unroll
        for (int x = 0; x < V; ++x) acc[x] = 0.f;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            // a split that saw no key has weight 0 and never wrote its partial output: what sits there is stale
            const float w = (lv[k] != ninf) ? ex2f(lv[k] - lse) : 0.f;
#pragma unroll
            for (int x = 0; x < V; ++x) acc[x] = (w != 0.f) ? fmaf(w, ov[k][x], acc[x]) : acc[x];
        }
        __nv_bfloat16 *dst = static_cast<__nv_bfloat16 *>(p.out) + rh * D + lane * V;
#pragma unroll
        for (int x = 0; x < V; x += 2)
            *reinterpret_cast<__nv_bfloat162 *>(dst + x) = __floats2bfloat162_rn(acc[x], acc[x + 1]);
        if (p.mass) {
            if (lane <= G) {
                float w = 0.f;
#pragma unroll
                for (int k = 0; k < 4; ++k) w += ex2f(sv[k] - lse_s);       // exp2(-inf) = 0: absent slots drop out
                p.mass[rh * p.mass_stride + lane] = w;
            }
            for (int s = lane + 32; s <= G; s += 32) {                      // more than 32 slots: the rest, as below
                float w = 0.f;
                for (int k = 0; k < p.n_splits; ++k) {
                    const float v = __ldcg(p.part_slot + (k * split_stride + rh) * p.slot_stride + s);
                    if (v != ninf) w += ex2f(v - lse);
                }
                p.mass[rh * p.mass_stride + s] = w;
            }
        }
        return;
    }

    // every lane needs every split's log-sum-exp: lane k loads split k (and k + 32), then shuffles
    float my0 = lane < p.n_splits ? p.part_lse[lane * split_stride + rh] : ninf;
    float my1 = lane + 32 < p.n_splits ? p.part_lse[(lane + 32) * split_stride + rh] : ninf;
    float mx = fmaxf(my0, my1);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    float sum = (my0 != ninf ? ex2f(my0 - mx) : 0.f) + (my1 != ninf ? ex2f(my1 - mx) : 0.f);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    const float lse = mx + log2f(sum);
    const float w0 = my0 != ninf ? ex2f(my0 - lse) : 0.f;
    const float w1 = my1 != ninf ? ex2f(my1 - lse) : 0.f;

    float acc[V];
#pragma unroll
    for (int x = 0; x < V; ++x) acc[x] = 0.f;
    for (int k = 0; k < p.n_splits; ++k) {
        const float w = __shfl_sync(0xffffffffu, k < 32 ? w0 : w1, k & 31);
        if (w != 0.f) {
            const float *src = p.part_o + (k * split_stride + rh) * D + lane * V;
            if constexpr (V == 4) {
                const float4 v = *reinterpret_cast<const float4 *>(src);
                acc[0] += w * v.x; acc[1] += w * v.y; acc[2] += w * v.z; acc[3] += w * v.w;
            } else {
                const float2 v = *reinterpret_cast<const float2 *>(src);
                acc[0] += w * v.x; acc[1] += w * v.y;
            }
        }
    }
    __nv_bfloat16 *dst = static_cast<__nv_bfloat16 *>(p.out) + rh * D + lane * V;
#pragma unroll
    for (int x = 0; x < V; x += 2)
        *reinterpret_cast<__nv_bfloat162 *>(dst + x) = __floats2bfloat162_rn(acc[x], acc[x + 1]);

    if (p.mass) {
        const int G = p.row_slots[row];
        for (int s = lane; s <= G; s += 32) {
            float w = 0.f;
            for (int k = 0; k < p.n_splits; ++k) {
                const float v = p.part_slot[(k * split_stride + rh) * p.slot_stride + s];
                if (v != ninf) w += ex2f(v - lse);
            }
            p.mass[rh * p.mass_stride + s] = w;
        }
    }
}

// grid (pairs, layers, 2): one CTA moves one page of K or V of one layer, 16 bytes per thread and trip
__global__ void page_copy_kernel(const uint8_t *src_k, const uint8_t *src_v, uint8_t *dst_k, uint8_t *dst_v,
                                 size_t src_layer_bytes, size_t dst_layer_bytes, const int2 *pairs, int page_bytes)
{
    pdl_trigger();
    pdl_wait();
    const int2 pr = pairs[blockIdx.x];
    const uint8_t *s = (blockIdx.z ? src_v : src_k) + src_layer_bytes * blockIdx.y + static_cast<size_t>(pr.x) * page_bytes;
    uint8_t *d = (blockIdx.z ? dst_v : dst_k) + dst_layer_bytes * blockIdx.y + static_cast<size_t>(pr.y) * page_bytes;
    for (int i = threadIdx.x * 16; i < page_bytes; i += blockDim.x * 16)
        *reinterpret_cast<uint4 *>(d + i) = *reinterpret_cast<const uint4 *>(s + i);
}

}  // namespace

cudaError_t launch_page_copy(const uint8_t *src_k, const uint8_t *src_v, uint8_t *dst_k, uint8_t *dst_v,
                             size_t src_layer_bytes, size_t dst_layer_bytes, const int2 *pairs, int n_pairs,
                             int n_layers, int page_bytes, cudaStream_t st)
{
    if (n_pairs <= 0) return cudaSuccess;
    const cudaError_t e = launch_pdl_n(page_copy_kernel, dim3(n_pairs, n_layers, 2), dim3(256), st, src_k, src_v, dst_k, dst_v,
                                       src_layer_bytes, dst_layer_bytes, pairs, page_bytes);
    return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t launch_page_scatter(void *kpool_layer, void *vpool_layer, const void *k, const void *v,
                                const PageRun &run, int first_pos, int n_tokens, int zero_rows, int Hkv, int D,
                                int n_sm, cudaStream_t st)
{
    if (n_tokens <= 0) return cudaSuccess;
    const int cpr = D * 2 / 16;
    const long long total = static_cast<long long>(n_tokens + zero_rows) * Hkv * cpr;
    const int threads = 256;
    long long blocks = (total + threads - 1) / threads;
    if (blocks > n_sm * 8) blocks = n_sm * 8;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(blocks));
    cfg.blockDim = dim3(threads);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, page_scatter_kernel, static_cast<uint4 *>(kpool_layer),
                                             static_cast<uint4 *>(vpool_layer), static_cast<const uint4 *>(k),
                                             static_cast<const uint4 *>(v), run, first_pos, n_tokens, zero_rows, Hkv, cpr);
    return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t launch_page_scatter_layers(void *kpool, void *vpool, size_t layer_bytes, int layer0, int n_layers,
                                       const LayerSrc &src, size_t src_off, const PageRun &run, int first_pos,
                                       int n_tokens, int zero_rows, int Hkv, int D, int n_sm, cudaStream_t st)
{
    if (n_tokens <= 0 || n_layers <= 0) return cudaSuccess;
    if (n_layers > kScatterLayers) return cudaErrorInvalidValue;
    const int cpr = D * 2 / 16;
    const long long total = static_cast<long long>(n_tokens + zero_rows) * Hkv * cpr;
    const int threads = 256;
    long long blocks = (total + threads - 1) / threads;
    const long long cap = std::max(1, n_sm * 8 / n_layers);
    if (blocks > cap) blocks = cap;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(blocks), static_cast<unsigned>(n_layers));
    cfg.blockDim = dim3(threads);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    uint4 *kp = reinterpret_cast<uint4 *>(static_cast<uint8_t *>(kpool) + layer_bytes * layer0);
    uint4 *vp = reinterpret_cast<uint4 *>(static_cast<uint8_t *>(vpool) + layer_bytes * layer0);
    const cudaError_t e = cudaLaunchKernelEx(&cfg, page_scatter_layers_kernel, kp, vp,
                                             static_cast<long long>(layer_bytes / 16), src,
                                             static_cast<long long>(src_off / 16), run, first_pos, n_tokens, zero_rows, Hkv, cpr);
    return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t launch_combine(const CombineParams &p, cudaStream_t st)
{
    const long long pairs = static_cast<long long>(p.n_q_total) * p.Hq;
    if (pairs <= 0) return cudaSuccess;
    const int warps = 8;
    const int blocks = static_cast<int>((pairs + warps - 1) / warps);
    const cudaError_t e = (p.D == 128) ? launch_pdl(combine_kernel<128>, dim3(blocks), dim3(warps * 32), 0, st, p)
                                       : launch_pdl(combine_kernel<64>, dim3(blocks), dim3(warps * 32), 0, st, p);
    return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace enl
