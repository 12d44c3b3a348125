// Clustering reduce (paper, Sec. 3.3 "Attention-based Memory Clustering"): the average attention between a
// newly detected object and every existing group, over the object's query tokens, all q heads and the few
// scored layers, and the decision: the object joins the group whose average exceeds the threshold, else it opens
// a new group.
// Input is the per-group mass that enl_attend returns for the scoring pass; this is the reduction that
// consumes it.  Bandwidth-bound: every mass value is read once, coalesced along the group axis.
#include <cuda_runtime.h>

#include "../../include/enl.h"
#include "enl_internal.h"

namespace {

constexpr int kMaxLayers = ENL_CLUSTER_MAX_LAYERS;
constexpr int kMaxObjects = ENL_CLUSTER_MAX_OBJECTS;
constexpr int kWarps = 8;
constexpr int kGroupsPerCta = 32;             // one group per lane
constexpr int kUnroll = 16;                   // (row, head) pairs, i.e. loads, in flight per warp

struct ClusterParams {
    const float *mass[kMaxLayers];
    int32_t obj_off[kMaxObjects + 1];
    int32_t n_layers, Hq, mass_stride, n_groups, n_obj;
    float threshold;
    float *avg;
    int32_t *assign;
};

// grid (objects, ceil(n_groups / 32)); warp w takes (row, head) pairs w, w + 8, ... of the object's span, lane l
// sums group l of the CTA's 32-group chunk: every warp load is one coalesced 128-byte line whatever the row
// stride, and sixteen of them are in flight per warp.  Many small CTAs (eight resident per SM) rather than few
// large ones: with equal-sized CTAs a second, partly filled wave would cost up to half the time.
__global__ void __launch_bounds__(kWarps * 32) cluster_avg_kernel(const __grid_constant__ ClusterParams p)
{
    __shared__ float part[kWarps][kGroupsPerCta];
    const int obj = blockIdx.x, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = blockIdx.y * kGroupsPerCta + lane;
    const int r0 = p.obj_off[obj], r1 = p.obj_off[obj + 1];
    const long long pairs = static_cast<long long>(r1 - r0) * p.Hq;
    enl::pdl_trigger();
    enl::pdl_wait();                                   // the masses come from the attention kernels before
    const bool on = g < p.n_groups;
    float acc = 0.f;
    for (int l = 0; l < p.n_layers; ++l) {
        const float *base = p.mass[l] + static_cast<long long>(r0) * p.Hq * p.mass_stride + g;
        long long i = warp;
        for (; i + (kUnroll - 1) * kWarps < pairs; i += kUnroll * kWarps) {
            float v[kUnroll];
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) v[u] = on ? __ldcs(base + (i + u * kWarps) * p.mass_stride) : 0.f;
            // summed in the order of the pairs, as a plain loop would
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) acc += v[u];
        }
        for (; i < pairs; i += kWarps)
            if (on) acc += __ldcs(base + i * p.mass_stride);
    }
    part[warp][lane] = acc;
    __syncthreads();
    if (warp == 0) {
        float t = 0.f;
        for (int w = 0; w < kWarps; ++w) t += part[w][lane];
        const float inv = (pairs > 0) ? 1.f / (static_cast<float>(pairs) * static_cast<float>(p.n_layers)) : 0.f;
        if (on) p.avg[static_cast<long long>(obj) * p.n_groups + g] = t * inv;
    }
}

// one warp per object: the group with the largest average (lowest index on ties); -1 unless it exceeds the threshold
__global__ void cluster_pick_kernel(const float *avg, int32_t *assign, int n_groups, int n_obj, float threshold)
{
    const int obj = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    enl::pdl_trigger();
    enl::pdl_wait();
    if (obj >= n_obj) return;
    float best = -1.f;
    int arg = -1;
    for (int g = lane; g < n_groups; g += 32) {
        const float v = avg[static_cast<long long>(obj) * n_groups + g];
        if (v > best) { best = v; arg = g; }
    }
    for (int o = 16; o > 0; o >>= 1) {
        const float ob = __shfl_xor_sync(0xffffffffu, best, o);
        const int oa = __shfl_xor_sync(0xffffffffu, arg, o);
        if (ob > best || (ob == best && oa >= 0 && (arg < 0 || oa < arg))) { best = ob; arg = oa; }
    }
    if (lane == 0) assign[obj] = (arg >= 0 && best > threshold) ? arg : -1;
}

// avg[o][g] = sum[o][g] / (rows of o * q heads * layers): the sums come out of the attention kernel itself
struct SumParams {
    int32_t obj_off[kMaxObjects + 1];
    const float *sum;
    float *avg;
    int32_t sum_stride, n_groups, n_obj;
    float per_row;                                     // 1 / (q heads * layers)
};
__global__ void cluster_scale_kernel(const __grid_constant__ SumParams p)
{
    const int obj = blockIdx.y;
    const int g = blockIdx.x * blockDim.x + threadIdx.x;
    enl::pdl_trigger();
    enl::pdl_wait();
    if (g >= p.n_groups) return;
    const int rows = p.obj_off[obj + 1] - p.obj_off[obj];
    const float inv = rows > 0 ? p.per_row / static_cast<float>(rows) : 0.f;
    p.avg[static_cast<long long>(obj) * p.n_groups + g] = p.sum[static_cast<long long>(obj) * p.sum_stride + g] * inv;
}

}  // namespace

extern "C" int enl_cluster_assign_sums(const float *mass_sum, int32_t sum_stride, int32_t n_groups, int32_t n_obj,
                                       const int32_t *obj_off, int32_t n_q_heads, int32_t n_layers, float threshold,
                                       float *avg, int32_t *assign, void *cuda_stream)
{
    if (!mass_sum || !obj_off || !avg || !assign) return ENL_E_INVAL;
    if (n_groups < 1 || n_obj < 1 || n_q_heads < 1 || n_layers < 1 || sum_stride < n_groups) return ENL_E_INVAL;
    if (n_obj > kMaxObjects) return ENL_E_LIMIT;
    SumParams p;
    if (obj_off[0] < 0) return ENL_E_INVAL;
    for (int o = 0; o <= n_obj; ++o) {
        if (o > 0 && obj_off[o] < obj_off[o - 1]) return ENL_E_INVAL;
        p.obj_off[o] = obj_off[o];
    }
    p.sum = mass_sum;
    p.avg = avg;
    p.sum_stride = sum_stride;
    p.n_groups = n_groups;
    p.n_obj = n_obj;
    p.per_row = 1.f / (static_cast<float>(n_q_heads) * static_cast<float>(n_layers));
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const dim3 grid((n_groups + 127) / 128, n_obj);
    if (enl::launch_pdl(cluster_scale_kernel, grid, dim3(128), 0, st, p) != cudaSuccess) { cudaGetLastError(); return ENL_E_CUDA; }
    if (enl::launch_pdl_n(cluster_pick_kernel, dim3((n_obj + 3) / 4), dim3(128), st, avg, assign, n_groups, n_obj, threshold) != cudaSuccess) {
        cudaGetLastError();
        return ENL_E_CUDA;
    }
    return ENL_OK;
}

extern "C" int enl_cluster_assign(const enl_cluster_args_t *a, void *cuda_stream)
{
    if (!a || !a->mass || !a->obj_off || !a->avg || !a->assign) return ENL_E_INVAL;
    if (a->n_layers < 1 || a->n_q < 1 || a->n_q_heads < 1 || a->n_groups < 1 || a->n_obj < 1) return ENL_E_INVAL;
    if (a->mass_stride < a->n_groups) return ENL_E_INVAL;
    if (a->n_layers > kMaxLayers || a->n_obj > kMaxObjects) return ENL_E_LIMIT;
    ClusterParams p;
    for (int l = 0; l < a->n_layers; ++l) {
        if (!a->mass[l] || (reinterpret_cast<uintptr_t>(a->mass[l]) & 3)) return ENL_E_INVAL;
        p.mass[l] = a->mass[l];
    }
    for (int l = a->n_layers; l < kMaxLayers; ++l) p.mass[l] = nullptr;
    if (a->obj_off[0] < 0) return ENL_E_INVAL;
    for (int o = 0; o <= a->n_obj; ++o) {
        if (o > 0 && a->obj_off[o] < a->obj_off[o - 1]) return ENL_E_INVAL;
        p.obj_off[o] = a->obj_off[o];
    }
    if (a->obj_off[a->n_obj] > a->n_q) return ENL_E_INVAL;
    p.n_layers = a->n_layers;
    p.Hq = a->n_q_heads;
    p.mass_stride = a->mass_stride;
    p.n_groups = a->n_groups;
    p.n_obj = a->n_obj;
    p.threshold = a->threshold;
    p.avg = a->avg;
    p.assign = a->assign;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const dim3 grid(a->n_obj, (a->n_groups + kGroupsPerCta - 1) / kGroupsPerCta);
    if (enl::launch_pdl(cluster_avg_kernel, grid, dim3(kWarps * 32), 0, st, p) != cudaSuccess) { cudaGetLastError(); return ENL_E_CUDA; }
    if (enl::launch_pdl_n(cluster_pick_kernel, dim3((a->n_obj + 3) / 4), dim3(128), st, a->avg, a->assign, a->n_groups,
                          a->n_obj, a->threshold) != cudaSuccess) {
        cudaGetLastError();
        return ENL_E_CUDA;
    }
    return ENL_OK;
}
