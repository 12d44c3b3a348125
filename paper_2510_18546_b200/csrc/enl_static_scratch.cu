// enl_attend_static: one-token selective-KV attention for callers that may not allocate device memory.
//
// The regular path keeps its split-KV partial results in scratch that enl_cache_create allocates.  Some
// callers cannot do that: a planner tick running inside a real-time control loop whose memory was fixed
// at start-up, a plug-in living inside another runtime that owns the whole device heap, a process whose
// CUDA allocator is locked down after initialisation.  For them this file offers the same split-KV
// computation (partial attention per key range, then the log-sum-exp merge) with the partials held in
// a file-scope device array of fixed size: no cudaMalloc, no cudaFree, no allocating library call,
// and no host heap allocation either.  Keys and values come as one contiguous caller-owned buffer
// instead of the paged pool, because the pool itself is something only an allocating caller can have.
//
// The device array's name is only a host-side handle in host code; its device address is looked up
// once per device with cudaGetSymbolAddress (the first call on that device does it) and handed to
// the kernels as an ordinary pointer.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "../../include/enl.h"
#include "enl_internal.h"

namespace {

constexpr int kMaxDevices   = 64;
constexpr int kMaxSeg       = ENL_STATIC_MAX_SEGMENTS;
constexpr int kMaxSplits    = 64;
constexpr int kKeysPerSplit = 1024;                              // scores of one split live in shared memory
constexpr int kMaxRep       = 8;                                 // q heads per kv head
constexpr int kThreads      = 128;
constexpr size_t kScratchBytes = ENL_STATIC_SCRATCH_BYTES;
constexpr size_t kHeaderBytes  = 256;                            // row -> slot count word for the merge kernel

// Partials of the last call stay here until the next call overwrites them; every entry a call reads
// is written by that call first, so nothing has to be cleared in between.
static __device__ __align__(256) unsigned char g_static_scratch[kScratchBytes];

struct SegTable {
    int32_t off[kMaxSeg + 2];          // off[s] = first key of slot s; slot n_seg = the new keys; off[n_seg + 1] = total
};

struct StaticParams {
    const __nv_bfloat16 *q, *k, *v;
    float *part_o, *part_lse, *part_slot;
    int32_t *row_slots;
    int32_t Hq, Hkv, rep, n_seg, n_splits, total_keys;
    float scale_log2;
};

__device__ __forceinline__ float ex2a(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// grid (n_splits, Hkv); the CTA covers keys [k0, k1) of the stream for the rep q heads of one kv head.
template <int D>
__global__ void __launch_bounds__(kThreads) static_partial_kernel(const StaticParams p, const __grid_constant__ SegTable seg)
{
    __shared__ float sc[kMaxRep][kKeysPerSplit];
    __shared__ float row_m[kMaxRep], row_l[kMaxRep];
    constexpr int V = D / 32;                                    // channels per lane
    const int split = blockIdx.x, kvh = blockIdx.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int k0 = static_cast<int>(static_cast<long long>(p.total_keys) * split / p.n_splits);
    const int k1 = static_cast<int>(static_cast<long long>(p.total_keys) * (split + 1) / p.n_splits);
    const int n = k1 - k0;
    const int rep = p.rep;
    const float ninf = -__builtin_huge_valf();
    if (split == 0 && kvh == 0 && threadIdx.x == 0) p.row_slots[0] = p.n_seg;

    // phase A: scores, one key per warp iteration, lanes over channels
    float qv[kMaxRep][V];
#pragma unroll
    for (int h = 0; h < kMaxRep; ++h)
#pragma unroll
        for (int x = 0; x < V; ++x)
            qv[h][x] = (h < rep) ? __bfloat162float(p.q[(kvh * rep + h) * D + lane * V + x]) : 0.f;
    for (int j = warp; j < n; j += kThreads / 32) {
        const __nv_bfloat16 *kr = p.k + (static_cast<long long>(k0 + j) * p.Hkv + kvh) * D + lane * V;
        float kx[V];
#pragma unroll
        for (int x = 0; x < V; ++x) kx[x] = __bfloat162float(kr[x]);
#pragma unroll
        for (int h = 0; h < kMaxRep; ++h) {
            if (h < rep) {
                float d = 0.f;
#pragma unroll
                for (int x = 0; x < V; ++x) d += qv[h][x] * kx[x];
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) d += __shfl_xor_sync(0xffffffffu, d, o);
                if (lane == 0) sc[h][j] = d * p.scale_log2;
            }
        }
    }
    __syncthreads();

    // phase B: per q head (one warp each) maximum, probabilities, per-slot sums
    const long long sh = static_cast<long long>(split) * p.Hq;    // one query row: [split][0][Hq]
    for (int h = warp; h < rep; h += kThreads / 32) {
        float m = ninf;
        for (int j = lane; j < n; j += 32) m = fmaxf(m, sc[h][j]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
        const float m_use = (m == ninf) ? 0.f : m;
        float l = 0.f;
        float *slot_out = p.part_slot ? p.part_slot + (sh + kvh * rep + h) * (p.n_seg + 1) : nullptr;
        for (int s = 0; s <= p.n_seg; ++s) {
            const int a = max(seg.off[s], k0), b = min(seg.off[s + 1], k1);
            float w = 0.f;
            for (int j = a + lane; j < b; j += 32) {
                const float e = ex2a(sc[h][j - k0] - m_use);
                sc[h][j - k0] = e;
                w += e;
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) w += __shfl_xor_sync(0xffffffffu, w, o);
            l += w;
            if (slot_out && lane == 0) slot_out[s] = (w > 0.f) ? log2f(w) + m_use : ninf;
        }
        if (lane == 0) {
            row_m[h] = m_use;
            row_l[h] = l;
            p.part_lse[sh + kvh * rep + h] = (l > 0.f) ? m_use + log2f(l) : ninf;
        }
    }
    __syncthreads();

    // phase C: partial output, one thread per channel
    if (threadIdx.x < D) {
        float acc[kMaxRep];
#pragma unroll
        for (int h = 0; h < kMaxRep; ++h) acc[h] = 0.f;
        const __nv_bfloat16 *vc = p.v + (static_cast<long long>(k0) * p.Hkv + kvh) * D + threadIdx.x;
        for (int j = 0; j < n; ++j) {
            const float vv = __bfloat162float(vc[static_cast<long long>(j) * p.Hkv * D]);
#pragma unroll
            for (int h = 0; h < kMaxRep; ++h)
                if (h < rep) acc[h] += sc[h][j] * vv;
        }
#pragma unroll
        for (int h = 0; h < kMaxRep; ++h)
            if (h < rep) {
                const float l = row_l[h];
                p.part_o[(sh + kvh * rep + h) * D + threadIdx.x] = (l > 0.f) ? acc[h] / l : 0.f;
            }
    }
}

// Device address of the static array, looked up once per device (with that device current).
cudaError_t scratch_address(unsigned char **out)
{
    static unsigned char *addr[kMaxDevices] = {};
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    unsigned char *p = __atomic_load_n(&addr[dev], __ATOMIC_ACQUIRE);
    if (!p) {
        void *sym = nullptr;
        e = cudaGetSymbolAddress(&sym, g_static_scratch);
        if (e != cudaSuccess) return e;
        p = static_cast<unsigned char *>(sym);
        __atomic_store_n(&addr[dev], p, __ATOMIC_RELEASE);      // racing first calls store the same value
    }
    *out = p;
    return cudaSuccess;
}

}  // namespace

extern "C" int enl_attend_static(const enl_static_args_t *a, void *cuda_stream)
{
    if (!a) return ENL_E_INVAL;
    if (a->n_q_heads <= 0 || a->n_kv_heads <= 0 || a->n_q_heads % a->n_kv_heads != 0) return ENL_E_INVAL;
    if (a->head_dim != 64 && a->head_dim != 128) return ENL_E_INVAL;
    if (a->n_seg < 0 || a->n_new < 1 || (a->n_seg > 0 && !a->seg_len)) return ENL_E_INVAL;
    if (!a->q || !a->k || !a->v || !a->out) return ENL_E_INVAL;
    const int rep = a->n_q_heads / a->n_kv_heads;
    if (rep > kMaxRep || a->n_seg > kMaxSeg) return ENL_E_LIMIT;

    SegTable seg;
    long long acc = 0;
    for (int s = 0; s < a->n_seg; ++s) {
        if (a->seg_len[s] < 0) return ENL_E_INVAL;
        seg.off[s] = static_cast<int32_t>(acc);
        acc += a->seg_len[s];
        if (acc > ENL_STATIC_MAX_KEYS) return ENL_E_LIMIT;
    }
    seg.off[a->n_seg] = static_cast<int32_t>(acc);
    acc += a->n_new;
    if (acc > ENL_STATIC_MAX_KEYS) return ENL_E_LIMIT;
    const int total = static_cast<int>(acc);
    for (int s = a->n_seg + 1; s < kMaxSeg + 2; ++s) seg.off[s] = total;

    // splits: enough that a split's scores fit shared memory, more while they keep the SMs busy, never more
    // than the static array can hold
    const size_t per_split = static_cast<size_t>(a->n_q_heads) * (a->head_dim + 1 + (a->group_mass ? a->n_seg + 1 : 0)) * sizeof(float);
    const int need = (total + kKeysPerSplit - 1) / kKeysPerSplit;
    const int fit = static_cast<int>((kScratchBytes - kHeaderBytes) / per_split);
    if (fit < need) return ENL_E_LIMIT;
    int want = (total + 255) / 256;
    if (want < need) want = need;
    if (want > kMaxSplits) want = kMaxSplits;
    const int n_splits = want < fit ? want : fit;

    unsigned char *base = nullptr;
    if (scratch_address(&base) != cudaSuccess) { cudaGetLastError(); return ENL_E_CUDA; }
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);

    StaticParams p;
    p.q = static_cast<const __nv_bfloat16 *>(a->q);
    p.k = static_cast<const __nv_bfloat16 *>(a->k);
    p.v = static_cast<const __nv_bfloat16 *>(a->v);
    const size_t rows = static_cast<size_t>(n_splits) * a->n_q_heads;
    p.row_slots = reinterpret_cast<int32_t *>(base);
    p.part_o = reinterpret_cast<float *>(base + kHeaderBytes);
    p.part_lse = p.part_o + rows * a->head_dim;
    p.part_slot = a->group_mass ? p.part_lse + rows : nullptr;
    p.Hq = a->n_q_heads;
    p.Hkv = a->n_kv_heads;
    p.rep = rep;
    p.n_seg = a->n_seg;
    p.n_splits = n_splits;
    p.total_keys = total;
    p.scale_log2 = 1.4426950408889634f / sqrtf(static_cast<float>(a->head_dim));

    const dim3 grid(n_splits, a->n_kv_heads);
    if (a->head_dim == 128) static_partial_kernel<128><<<grid, kThreads, 0, st>>>(p, seg);
    else static_partial_kernel<64><<<grid, kThreads, 0, st>>>(p, seg);
    if (cudaGetLastError() != cudaSuccess) return ENL_E_CUDA;

    enl::CombineParams cp;
    cp.part_o = p.part_o;
    cp.part_lse = p.part_lse;
    cp.part_slot = p.part_slot;
    cp.out = a->out;
    cp.mass = a->group_mass;
    cp.row_slots = p.row_slots;
    cp.n_q_total = 1;
    cp.Hq = a->n_q_heads;
    cp.D = a->head_dim;
    cp.slot_stride = a->n_seg + 1;
    cp.mass_stride = a->n_seg + 1;
    cp.n_splits = n_splits;
    if (enl::launch_combine(cp, st) != cudaSuccess) { cudaGetLastError(); return ENL_E_CUDA; }
    return ENL_OK;
}
