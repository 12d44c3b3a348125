// Small kernels around the attention: scatter of a group's K/V rows into pool pages (the store of
// Sec. 3.2 "Discrete Memory Caching") and the merge of KV splits (log-sum-exp weighted average of the
// partial outputs, sum of the partial per-slot masses).
#include <cuda_bf16.h>

#include "enl_internal.h"

namespace enl {
namespace {

// k, v: [n_tokens][Hkv][D] bf16 -> pool layer [page][Hkv][16][D]; 16-byte chunks, one per thread-iteration.
__global__ void page_scatter_kernel(uint4 *__restrict__ kpool, uint4 *__restrict__ vpool,
                                    const uint4 *__restrict__ k, const uint4 *__restrict__ v,
                                    const __grid_constant__ PageRun run, int first_pos, int n_tokens,
                                    int Hkv, int chunks_per_row)
{
    const long long total = static_cast<long long>(n_tokens) * Hkv * chunks_per_row;
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
        kpool[dst] = k[id];
        vpool[dst] = v[id];
    }
}

__device__ __forceinline__ float ex2f(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// One block per (query row, q head); thread d merges channel d, then the threads stride over the slots.
__global__ void combine_kernel(const CombineParams p)
{
    const long long rh = blockIdx.x;                       // row * Hq + head
    const int row = static_cast<int>(rh / p.Hq);
    const long long split_stride = static_cast<long long>(p.n_q_total) * p.Hq;
    const float ninf = -__builtin_huge_valf();

    float mx = ninf;
    for (int k = 0; k < p.n_splits; ++k) mx = fmaxf(mx, p.part_lse[k * split_stride + rh]);
    float sum = 0.f;
    for (int k = 0; k < p.n_splits; ++k) {
        const float v = p.part_lse[k * split_stride + rh];
        if (v != ninf) sum += ex2f(v - mx);
    }
    const float lse = mx + log2f(sum);

    for (int d = threadIdx.x; d < p.D; d += blockDim.x) {
        float o = 0.f;
        for (int k = 0; k < p.n_splits; ++k) {
            const float v = p.part_lse[k * split_stride + rh];
            if (v != ninf) o += ex2f(v - lse) * p.part_o[(k * split_stride + rh) * p.D + d];
        }
        static_cast<__nv_bfloat16 *>(p.out)[rh * p.D + d] = __float2bfloat16_rn(o);
    }
    if (p.mass) {
        const int G = p.row_slots[row];
        for (int s = threadIdx.x; s <= G; s += blockDim.x) {
            float w = 0.f;
            for (int k = 0; k < p.n_splits; ++k) {
                const float v = p.part_slot[(k * split_stride + rh) * p.slot_stride + s];
                if (v != ninf) w += ex2f(v - lse);
            }
            p.mass[rh * p.mass_stride + s] = w;
        }
    }
}

}  // namespace

cudaError_t launch_page_scatter(void *kpool_layer, void *vpool_layer, const void *k, const void *v,
                                const PageRun &run, int first_pos, int n_tokens, int Hkv, int D,
                                cudaStream_t st)
{
    if (n_tokens <= 0) return cudaSuccess;
    const int cpr = D * 2 / 16;
    const long long total = static_cast<long long>(n_tokens) * Hkv * cpr;
    const int threads = 256;
    long long blocks = (total + threads - 1) / threads;
    if (blocks > 148 * 8) blocks = 148 * 8;
    page_scatter_kernel<<<static_cast<int>(blocks), threads, 0, st>>>(
        static_cast<uint4 *>(kpool_layer), static_cast<uint4 *>(vpool_layer), static_cast<const uint4 *>(k),
        static_cast<const uint4 *>(v), run, first_pos, n_tokens, Hkv, cpr);
    return cudaGetLastError();
}

cudaError_t launch_combine(const CombineParams &p, cudaStream_t st)
{
    const long long blocks = static_cast<long long>(p.n_q_total) * p.Hq;
    if (blocks <= 0) return cudaSuccess;
    combine_kernel<<<static_cast<int>(blocks), 128, 0, st>>>(p);
    return cudaGetLastError();
}

}  // namespace enl
