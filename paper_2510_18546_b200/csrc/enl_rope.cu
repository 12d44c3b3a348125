// Rotary position encoding of bf16 rows, in place (an optional helper; the attention path rotates nothing).
// Paper, Sec. 3.2: positions are encoded as in the cited rotary embedding and every group keeps the positions it
// was computed with.  Formula as published (Su et al., "RoFormer"): pair j of a head is turned by pos * base^(-2j/D).
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cmath>

#include "../../include/enl.h"
#include "enl_internal.h"

namespace {

constexpr int kMaxPairs = ENL_ROPE_MAX_HEAD_DIM / 2;

struct RopeParams {
    double inv_freq[kMaxPairs];       // base^(-2j/D), formed on the host in double
    __nv_bfloat16 *rows;
    const int32_t *positions;
    long long n_pairs_total;          // n * n_heads * D / 2
    int32_t n_heads, D, first_pos, interleaved;
};

// one thread per (row, head, pair)
__global__ void rope_kernel(const __grid_constant__ RopeParams p)
{
    const long long idx = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x;
    enl::pdl_trigger();
    enl::pdl_wait();                                   // the rows may come from the kernel before
    if (idx >= p.n_pairs_total) return;
    const int half = p.D / 2;
    const int j = static_cast<int>(idx % half);
    const long long rh = idx / half;                   // (row, head)
    const long long row = rh / p.n_heads;
    const int pos = p.positions ? p.positions[row] : p.first_pos + static_cast<int>(row);
    // the angle in double, brought into [-pi, pi] before it is rounded to fp32: positions reach 1e5 and more
    const double two_pi = 6.283185307179586476925286766559;
    double ang = static_cast<double>(pos) * p.inv_freq[j];
    ang -= two_pi * rint(ang / two_pi);
    float sn, cs;
    sincosf(static_cast<float>(ang), &sn, &cs);
    __nv_bfloat16 *base = p.rows + rh * p.D;
    const int i1 = p.interleaved ? 2 * j : j, i2 = p.interleaved ? 2 * j + 1 : j + half;
    const float x1 = __bfloat162float(base[i1]), x2 = __bfloat162float(base[i2]);
    base[i1] = __float2bfloat16_rn(x1 * cs - x2 * sn);
    base[i2] = __float2bfloat16_rn(x2 * cs + x1 * sn);
}

}  // namespace

extern "C" int enl_rope_rotate(void *rows, int32_t n, int32_t n_heads, int32_t head_dim, const int32_t *positions,
                               int32_t first_pos, double base, int32_t interleaved, void *cuda_stream)
{
    if (!rows || n < 0 || n_heads < 1 || head_dim < 2 || (head_dim & 1) || !(base > 0.0)) return ENL_E_INVAL;
    if (reinterpret_cast<uintptr_t>(rows) & 3) return ENL_E_INVAL;
    if (head_dim > ENL_ROPE_MAX_HEAD_DIM) return ENL_E_LIMIT;
    if (n == 0) return ENL_OK;
    RopeParams p;
    for (int j = 0; j < kMaxPairs; ++j)
        p.inv_freq[j] = j < head_dim / 2 ? std::pow(base, -2.0 * j / head_dim) : 0.0;
    p.rows = static_cast<__nv_bfloat16 *>(rows);
    p.positions = positions;
    p.n_pairs_total = static_cast<long long>(n) * n_heads * (head_dim / 2);
    p.n_heads = n_heads;
    p.D = head_dim;
    p.first_pos = first_pos;
    p.interleaved = interleaved ? 1 : 0;
    const int threads = 256;
    const long long blocks = (p.n_pairs_total + threads - 1) / threads;
    if (blocks > 0x7fffffffll) return ENL_E_LIMIT;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (enl::launch_pdl(rope_kernel, dim3(static_cast<unsigned>(blocks)), dim3(threads), 0, st, p) != cudaSuccess) {
        cudaGetLastError();
        return ENL_E_CUDA;
    }
    return ENL_OK;
}
