// Split-KV attention for one-token decode steps, sm_100a: an HBM-streaming kernel.
//
// What it computes (paper, App. A: decoding attends with the one new query over the concatenated K/V;
// Sec. 3.2: the cached part is the selected groups' K/V; Sec. 3.3: per-group attention mass): for one
// episode, one kv head and one range of the episode's key stream (16-token pages of the selected groups
// in list order, then the new-token keys), the partial attention of the rep q heads that read this kv
// head -- partial output normalised by the range's own sum, the range's log2-sum-exp and a per-slot
// log2-sum-exp -- which the split merge at the end of the kernel turns into the output row and the group masses.
//
// Every K and V page is read from HBM exactly once.  The CTA's 12 warps take its pages one at a time from a
// shared counter (a warp that is served faster by the memory system simply takes more pages: with fixed runs
// the first warp finished 6-7 us before the last); each warp has a private pair of TMA stages (one page of one
// head = 16 rows x D bf16, 128-byte swizzle) fed by its lane 0: K and V of the page it works on, refilled with
// the page it took next as soon as they are read.  Per page, all in registers:
//   S = Q K^T      mma.sync, A = the rep query rows padded to 16, B = the K page (ldmatrix)
//   p = exp2(S-m)  running maximum per head kept by the warp, O and the sums rescaled when it grows
//   O += P V       mma.sync, A = P straight from the S accumulators, B = the V page (ldmatrix.trans)
// A page belongs to one slot (a selected group, or the new tokens) and a warp's pages come in stream order, so
// its slot sums are running sums that are parked (slot id + log2 value, in a list of the CTA) whenever the slot
// changes.  No CTA barrier inside the stream.
// At the end the warps are merged through shared memory; with several splits the CTA that finishes
// last for its (episode, kv head) merges the splits' partial results (a counter per pair, reset by
// that CTA), so a decode step is one launch.
// The arithmetic intensity is 4 flop per byte, so the tensor work is noise; the roof is HBM bandwidth.
// Code outside the streaming loop runs once per CTA from a cold instruction cache (the K/V stream has
// pushed it out of L2 since the last launch), so those loops are kept rolled: their size is their cost.
#include <cuda_bf16.h>

#include "enl_internal.h"

namespace enl {
namespace {

constexpr int kWarps   = 12;                              // one CTA per SM; 384 threads leave 168 registers each
constexpr int kThreads = kWarps * 32;
constexpr int kStages  = 2;                               // TMA stages per warp: K and V of one page; 96 KB in flight per SM (D = 128)
constexpr int kMaxRep  = 8;                               // q heads per kv head (rows 8..15 of the MMA stay zero)
constexpr int kMaxEnt  = kDecodeMaxPages + kWarps;        // parked slot sums of a CTA: at most one per page and one more per warp
constexpr int kPrefetchPages = 48;                        // pages per CTA asked into the L2 before the previous kernel has ended
constexpr float kRescaleThreshold = 8.0f;                 // log2 units
constexpr unsigned long long kWaitLimitNs = 1000ull * 1000ull * 1000ull;

__device__ __forceinline__ uint32_t smem_u32(const void *p)
{
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// One poll: the thread may stay suspended inside the instruction for up to the hinted time, and is woken when
// the phase completes; a longer hint means fewer polling instructions competing with the warps that work.
constexpr uint32_t kSuspendHintNs = 20000;
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity), "r"(kSuspendHintNs) : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait, warp-uniform result.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, int32_t *status)
{
    bool ok = mbar_try_wait(bar, parity);
    if (!ok) {
        // the clock is read only every 16 failed polls (the first reading starts the limit): a poll already
        // sleeps inside the instruction
        unsigned long long t0 = 0;
        uint32_t spins = 0;
        while (!(ok = mbar_try_wait(bar, parity))) {
            if ((++spins & 15u) == 0u) {
                if (*abort_flag) break;
                const unsigned long long now = global_ns();
                if (t0 == 0) {
                    t0 = now;
                } else if (now - t0 > kWaitLimitNs) {
                    *abort_flag = 1;
                    atomicExch(status, 2);
                    break;
                }
            }
        }
    }
    return __all_sync(0xffffffffu, ok);
}
// The K/V stream is read once: its lines are marked evict-first so that what is reused from launch to launch
// (code, plan, partial results) stays in L2.
__device__ __forceinline__ uint64_t policy_evict_first()
{
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *tm, int x, int y, uint32_t bar, uint64_t pol)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;"
        ::"r"(dst), "l"(tm), "r"(x), "r"(y), "r"(bar), "l"(pol) : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *tm, int x, int y, int z, uint32_t bar,
                                            uint64_t pol)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3, %4}], [%5], %6;"
        ::"r"(dst), "l"(tm), "r"(x), "r"(y), "r"(z), "r"(bar), "l"(pol) : "memory");
}
// Brings a box into the L2 without a destination in the SM: it observes nothing, so it may run before the wait for
// the previous kernel of the stream (the L2 is the point of coherence: a later write to those lines updates them).
__device__ __forceinline__ void tma_prefetch_2d(const CUtensorMap *tm, int x, int y)
{
    asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global.tile [%0, {%1, %2}];" ::"l"(tm), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t (&r)[4])
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t addr, uint32_t (&r)[4])
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
// D (fp32, m16n8) += A (bf16, m16k16, row) * B (bf16, k16n8, col).  Rows 8..15 of A are always zero here, so
// the accumulators of those rows (z0, z1) stay zero and one pair serves every product.
__device__ __forceinline__ void mma_bf16(float &d0, float &d1, float &z0, float &z1, uint32_t a0, uint32_t a2,
                                         uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
        : "+f"(d0), "+f"(d1), "+f"(z0), "+f"(z1)
        : "r"(a0), "r"(0u), "r"(a2), "r"(0u), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float lg2(float x)
{
    float y;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float rcp(float x)
{
    float y;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    const __nv_bfloat162 b = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t *>(&b);
}

constexpr float kNegInf = -__builtin_huge_valf();

// Shared memory: [ring: warp][stage][D*32 B] | parked slot sums | the CTA's page list | slot table | per-warp (m, l) | split weights | barriers
template <int D>
struct DecCfg {
    static constexpr int kStageBytes = D * kPageTokens * 2;            // one page of one head: 4 KB (D=128) / 2 KB
    static constexpr int kRingBytes  = kWarps * kStages * kStageBytes;
    static constexpr int kEntOff     = kRingBytes;                     // [kMaxEnt][kMaxRep] float, then [kMaxEnt] slot ids
    static constexpr int kEntBytes   = kMaxEnt * (kMaxRep + 1) * 4;
    static constexpr int kListOff    = kEntOff + kEntBytes;            // [kDecodeMaxPages] (page id, slot << 8 | valid keys)
    static constexpr int kListBytes  = kDecodeMaxPages * 8;
    static constexpr int kCslotOff   = kListOff + kListBytes;          // [kDecodeMaxPages + 1][kMaxRep] slot sums
    static constexpr int kCslotBytes = (kDecodeMaxPages + 1) * kMaxRep * 4;
    static constexpr int kMiscOff    = kCslotOff + kCslotBytes;
    // wm[warp][rep], wl[warp][rep], counters[2 * kWarps], cm[rep], cl[rep], weights[rep][kMaxSplits], flags[4],
    // slot ranges of the splits [kMaxSplits] x (first, count)
    static constexpr int kMiscBytes  = (2 * kWarps * kMaxRep + 2 * kWarps + 2 * kMaxRep + kMaxRep * kMaxSplits + 4 + 2 * kMaxSplits) * 4;
    static constexpr int kBarOff     = (kMiscOff + kMiscBytes + 15) & ~15;
    static constexpr int kSmemBytes  = kBarOff + kWarps * kStages * 8 + 1024;   // + alignment slack
};

template <int D>
__global__ void __launch_bounds__(kThreads, 1) decode_kernel(const __grid_constant__ DecodeParams p)
{
    using C = DecCfg<D>;
    constexpr int kChunks = D / 8;                        // 16-byte chunks per row
    constexpr int kHalves = D / 64;                       // TMA boxes (64 channels) per page
    constexpr int kNB     = D / 8;                        // n-blocks of the PV product
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t sbase = (raw + 1023u) & ~1023u;
    uint8_t *smem = smem_raw + (sbase - raw);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, tq = lane & 3;               // MMA row group and thread-in-group
    float *ent_val = reinterpret_cast<float *>(smem + C::kEntOff);            // [kMaxEnt][kMaxRep]: parked log2 slot sums
    int *ent_slot = reinterpret_cast<int *>(ent_val + kMaxEnt * kMaxRep);     // [kMaxEnt]: their slots
    int2 *pg_list = reinterpret_cast<int2 *>(smem + C::kListOff);             // the CTA's pages in stream order
    float *cslot = reinterpret_cast<float *>(smem + C::kCslotOff);            // [slot][kMaxRep]: sum of shares, then log2-sum
    float *wm = reinterpret_cast<float *>(smem + C::kMiscOff);                // [warp][kMaxRep]
    float *wl = wm + kWarps * kMaxRep;
    int *ctrs = reinterpret_cast<int *>(wl + kWarps * kMaxRep);               // [0] next page to hand out, [1] parked entries
    float *cm = reinterpret_cast<float *>(ctrs + 2 * kWarps);                 // CTA (later: merged) log2-sum-exp reference
    float *cl = cm + kMaxRep;
    float *weights = cl + kMaxRep;                                            // [kMaxRep][kMaxSplits]
    volatile int *flags = reinterpret_cast<volatile int *>(weights + kMaxRep * kMaxSplits);   // [0] abort, [1] last
    volatile int *abort_flag = flags;
    int2 *rng_tab = reinterpret_cast<int2 *>(const_cast<int *>(flags) + 4);   // [split]: first slot and slots of its page range
    const uint32_t bar0 = sbase + C::kBarOff;
    auto bar_full = [&](int s) { return bar0 + 8u * (warp * kStages + s); };
    auto stage_addr = [&](int s) { return sbase + static_cast<uint32_t>((warp * kStages + s) * C::kStageBytes); };

    // grid = (splits, kv heads, episodes); a single episode travels in the parameters
    struct { int ep, kvh, split; } it = {static_cast<int>(blockIdx.z), static_cast<int>(blockIdx.y), static_cast<int>(blockIdx.x)};
    EpInfo ep;
    if (gridDim.z == 1) {
        ep = p.ep0;
    } else {
        const int4 *src = reinterpret_cast<const int4 *>(p.eps + it.ep);
        const int4 e0 = __ldg(src), e1 = __ldg(src + 1);
        ep.stream_off = e0.x; ep.n_ctiles = e0.y; ep.n_slots = e0.z; ep.q_off = e0.w;
        ep.n_q = e1.x; ep.new_off = e1.y; ep.n_new = e1.z; ep.pad = e1.w;
    }
    if (threadIdx.x == 0) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(&p.tm_kpool) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&p.tm_vpool) : "memory");
    }
    const int rep = p.rep;
    const int n_cached = ep.n_ctiles * kPagesPerTile;                         // cached stream entries (padded)
    const int n_newp = (ep.n_new + kPageTokens - 1) / kPageTokens;            // pages of new-token keys
    const int total = n_cached + n_newp;
    const int pg_beg = static_cast<int>(static_cast<long long>(total) * it.split / p.n_splits);
    const int pg_end = static_cast<int>(static_cast<long long>(total) * (it.split + 1) / p.n_splits);
    const int n_cta = pg_end - pg_beg;                                        // <= kDecodeMaxPages (host guarantees)
    const int G = ep.n_slots;

    auto entry_meta = [&](int e) -> int {                                     // slot << 8 | valid keys
        if (e < n_cached) return __ldg(p.stream_meta + ep.stream_off + e);
        const int i = e - n_cached;
        return (G << 8) | min(kPageTokens, ep.n_new - i * kPageTokens);
    };

    if (threadIdx.x == 0) { flags[0] = 0; flags[1] = 0; ctrs[0] = kWarps; ctrs[1] = 0; }
    // The slot range of every split of this (episode, kv head), from the plan (the same arithmetic as that split's
    // CTA uses): whichever CTA merges the splits at the end then needs no memory round trip to learn where each
    // split's slot sums lie.
    if (static_cast<int>(threadIdx.x) < p.n_splits && p.n_splits > 1) {
        const int k = threadIdx.x;
        const int b0 = static_cast<int>(static_cast<long long>(total) * k / p.n_splits);
        const int b1 = static_cast<int>(static_cast<long long>(total) * (k + 1) / p.n_splits);
        int2 r = make_int2(0, 0);
        if (b1 > b0) {
            const int s0 = entry_meta(b0) >> 8;
            r = make_int2(s0, (entry_meta(b1 - 1) >> 8) - s0 + 1);
        }
        rng_tab[k] = r;
    }
    // the CTA's page list (page id, slot << 8 | valid keys): one coalesced load up front, so that no global load
    // sits between a stage becoming free and its refill
    for (int i = threadIdx.x; i < n_cta; i += kThreads) {
        const int e = pg_beg + i;
        int2 w;
        if (e < n_cached) {
            w.x = __ldg(p.stream_page + ep.stream_off + e);
            w.y = __ldg(p.stream_meta + ep.stream_off + e);
        } else {
            w.x = -1 - (e - n_cached);                                       // new-token page, counted from the end
            w.y = entry_meta(e);
        }
        pg_list[i] = w;
    }
    if (lane == 0) {
        for (int s = 0; s < kStages; ++s) mbar_init(bar_full(s), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    pdl_trigger();
    // While the previous kernel of the stream drains (its CTAs merge their warps and splits for several microseconds
    // after their streams have ended, and HBM idles meanwhile), ask the first pages of this CTA's range into the L2:
    // the stream below then starts on hits.
    {
        const int n_pf = min(n_cta, kPrefetchPages);
        for (int i = threadIdx.x; i < n_pf * 2 * kHalves; i += kThreads) {
            const int pg = pg_list[i / (2 * kHalves)].x;
            const int r = i % (2 * kHalves);
            if (pg >= 0)
                tma_prefetch_2d(r >= kHalves ? &p.tm_vpool : &p.tm_kpool, (r % kHalves) * 64, (pg * p.Hkv + it.kvh) * kPageTokens);
        }
    }

    // ... and the query rows of this kv head (rep x D bf16, contiguous): whatever the kernel before writes there, the
    // L2 holds the current data, and the loads after the wait then need not go to HBM before the first S
    {
        const uint8_t *qb = reinterpret_cast<const uint8_t *>(p.q) +
                            (static_cast<long long>(ep.q_off) * p.Hq + it.kvh * rep) * D * 2;
        const int q_bytes = rep * D * 2;
        if (static_cast<int>(threadIdx.x) * 128 < q_bytes)
            asm volatile("prefetch.global.L2 [%0];" ::"l"(qb + threadIdx.x * 128) : "memory");
    }

    // so far only shared memory and the gather plan were touched; the caller's tensors and the pool come next
    pdl_wait();
    const uint64_t pol = policy_evict_first();
    // K (stage 0) or V (stage 1) of one page into this warp's ring
    auto issue = [&](bool is_v, int page) {
        const int st = is_v ? 1 : 0;
        const uint32_t full = bar_full(st), dst = stage_addr(st);
        mbar_expect_tx(full, static_cast<uint32_t>(C::kStageBytes));
        if (page >= 0) {
            const CUtensorMap *tm = is_v ? &p.tm_vpool : &p.tm_kpool;
            const int row = (page * p.Hkv + it.kvh) * kPageTokens;
#pragma unroll
            for (int hf = 0; hf < kHalves; ++hf) tma_load_2d(dst + hf * (kPageTokens * 128), tm, hf * 64, row, full, pol);
        } else {
            const CUtensorMap *tm = is_v ? &p.tm_vnew : &p.tm_knew;
            const int krow = ep.new_off + (-1 - page) * kPageTokens;         // rows past the tensor's end read as zero
#pragma unroll
            for (int hf = 0; hf < kHalves; ++hf)
                tma_load_3d(dst + hf * (kPageTokens * 128), tm, hf * 64, it.kvh, krow, full, pol);
        }
    };
    // the next page of the CTA that nobody has taken yet (CTA-relative index; >= n_cta: none left)
    auto claim = [&]() -> int {
        int v = 0;
        if (lane == 0) v = atomicAdd(&ctrs[0], 1);
        return __shfl_sync(0xffffffffu, v, 0);
    };
    int cur = warp;                                                          // the first round is handed out statically
    if (cur < n_cta && lane == 0) {
        const int pg = pg_list[cur].x;
        issue(false, pg);
        issue(true, pg);
    }
    int nxt = claim();

    // the query rows of this kv head as the A operand of S = Q K^T (rows >= rep stay zero)
    uint32_t qa[D / 16][2];
    {
        const __nv_bfloat16 *qrow = static_cast<const __nv_bfloat16 *>(p.q) +
                                    (static_cast<long long>(ep.q_off) * p.Hq + it.kvh * rep + g) * D;
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
            qa[ks][0] = (g < rep) ? *reinterpret_cast<const uint32_t *>(qrow + ks * 16 + 2 * tq) : 0u;
            qa[ks][1] = (g < rep) ? *reinterpret_cast<const uint32_t *>(qrow + ks * 16 + 8 + 2 * tq) : 0u;
        }
    }
    // Touch, while the first pages are on their way, every kernel parameter that is otherwise first read
    // after the stream: a miss in the constant cache costs about a microsecond, and there it would be exposed.
    asm volatile("" ::"l"(p.part_o), "l"(p.part_lse), "l"(p.part_slot), "l"(p.part_rng), "l"(p.counters), "l"(p.out),
                 "l"(p.mass), "r"(p.n_q_total), "r"(p.mass_stride), "r"(p.slot_stride), "r"(p.n_splits), "r"(p.Hq));
    const float scale = p.scale_log2;
    bool ok = true;
    int n_done = 0;                                                          // pages this warp has worked through

    // called by the whole warp after it has read the K or the V stage for the last time: the page taken next
    auto refill = [&](bool is_v) {
        __syncwarp();                                                        // orders the warp's reads before the copy
        if (lane == 0 && nxt < n_cta) {
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            issue(is_v, pg_list[nxt].x);
        }
    };

    float o[kNB][2];
#pragma unroll
    for (int nb = 0; nb < kNB; ++nb) { o[nb][0] = o[nb][1] = 0.f; }
    float z0 = 0.f, z1 = 0.f;               // accumulators of the unused MMA rows 8..15
    float m = kNegInf;                      // running reference maximum of row g (same in the four lanes of a quad)
    float lsum = 0.f, acc = 0.f;            // lane-local parts of the row sum and of the current slot's sum
    int cur_slot = -1;
    auto park = [&]() {                      // the slot that ends: its id and the log2 of its sum (absolute) join the CTA's list
        float a = acc;
        a += __shfl_xor_sync(0xffffffffu, a, 1);
        a += __shfl_xor_sync(0xffffffffu, a, 2);
        if (cur_slot >= 0) {
            int e = 0;
            if (lane == 0) { e = atomicAdd(&ctrs[1], 1); ent_slot[e] = cur_slot; }
            e = __shfl_sync(0xffffffffu, e, 0);
            if (tq == 0 && g < kMaxRep) ent_val[e * kMaxRep + g] = (a > 0.f) ? lg2(a) + m : kNegInf;
        }
        acc = 0.f;
    };

    for (; cur < n_cta && ok; ++n_done) {
        // ---- S = Q K^T ----
        ok = mbar_wait(bar_full(0), static_cast<uint32_t>(n_done & 1), abort_flag, p.status);
        if (!ok) break;
        uint32_t base = stage_addr(0);
        float c[2][2] = {{0.f, 0.f}, {0.f, 0.f}};
#pragma unroll
        for (int nb = 0; nb < 2; ++nb) {
            const int row = nb * 8 + (lane & 7);                             // token whose 16-byte chunks this lane addresses
#pragma unroll
            for (int kq = 0; kq < kChunks / 4; ++kq) {                       // four 8-channel chunks = two k16 steps
                const int ch = kq * 4 + (lane >> 3);
                const uint32_t addr = base + (ch >> 3) * (kPageTokens * 128) + row * 128 + (((ch & 7) ^ (row & 7)) << 4);
                uint32_t b[4];
                ldsm_x4(addr, b);
                mma_bf16(c[nb][0], c[nb][1], z0, z1, qa[2 * kq][0], qa[2 * kq][1], b[0], b[1]);
                mma_bf16(c[nb][0], c[nb][1], z0, z1, qa[2 * kq + 1][0], qa[2 * kq + 1][1], b[2], b[3]);
            }
        }
        const int meta = pg_list[cur].y;
        const int nv = meta & 0xff, slot = meta >> 8;
        const float s0 = (2 * tq < nv) ? c[0][0] * scale : kNegInf;
        const float s1 = (2 * tq + 1 < nv) ? c[0][1] * scale : kNegInf;
        const float s2 = (8 + 2 * tq < nv) ? c[1][0] * scale : kNegInf;
        const float s3 = (8 + 2 * tq + 1 < nv) ? c[1][1] * scale : kNegInf;
        refill(false);

        // ---- p = exp2(S - m), sums ----
        float mx = fmaxf(fmaxf(s0, s1), fmaxf(s2, s3));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        if (slot != cur_slot) { park(); cur_slot = slot; }
        if (__any_sync(0xffffffffu, mx > m + kRescaleThreshold)) {           // also when m is still -inf
            const float m_new = fmaxf(m, mx);
            const float alpha = (m == kNegInf) ? 0.f : ex2(m - m_new);      // nothing accumulated yet when m = -inf
            if (m_new != m) {
                lsum *= alpha;
                acc *= alpha;
            }
            // rows g (o[.][0..1]) scale by this lane's alpha; rows g + 8 hold only zeros
            const float a_row = (m_new != m) ? alpha : 1.f;
#pragma unroll
            for (int nb = 0; nb < kNB; ++nb) { o[nb][0] *= a_row; o[nb][1] *= a_row; }
            m = m_new;
        }
        const float m_use = (m == kNegInf) ? 0.f : m;
        const float p0 = ex2(s0 - m_use), p1 = ex2(s1 - m_use), p2 = ex2(s2 - m_use), p3 = ex2(s3 - m_use);
        const float ps = (p0 + p1) + (p2 + p3);
        acc += ps;
        lsum += ps;
        const uint32_t a0 = pack_bf16(p0, p1), a2 = pack_bf16(p2, p3);

        // ---- O += P V ----
        ok = mbar_wait(bar_full(1), static_cast<uint32_t>(n_done & 1), abort_flag, p.status);
        if (!ok) break;
        base = stage_addr(1);
        const int row = ((lane >> 3) & 1) * 8 + (lane & 7);                  // token addressed by this lane
#pragma unroll
        for (int nq = 0; nq < kNB / 2; ++nq) {                               // two 8-channel n-blocks per ldmatrix
            const int ch = nq * 2 + (lane >> 4);
            const uint32_t addr = base + (ch >> 3) * (kPageTokens * 128) + row * 128 + (((ch & 7) ^ (row & 7)) << 4);
            uint32_t b[4];
            ldsm_x4_trans(addr, b);
            mma_bf16(o[2 * nq][0], o[2 * nq][1], z0, z1, a0, a2, b[0], b[1]);
            mma_bf16(o[2 * nq + 1][0], o[2 * nq + 1][1], z0, z1, a0, a2, b[2], b[3]);
        }
        refill(true);
        cur = nxt;
        if (cur < n_cta) nxt = claim();
    }
    park();

    // error path only: give this warp's copies in flight (at most two pages) time to land before the CTA retires
    if (!ok && warp < n_cta) {
        const unsigned long long t0 = global_ns();
        while (global_ns() - t0 < 50000ull) { }
    }
    lsum += __shfl_xor_sync(0xffffffffu, lsum, 1);
    lsum += __shfl_xor_sync(0xffffffffu, lsum, 2);
    if (tq == 0) { wm[warp * kMaxRep + g] = m; wl[warp * kMaxRep + g] = lsum; }
    // slots the CTA's range touched, and their table cleared for the merge of the parked sums
    int slot_first = 0, n_local = 0;
    if (n_cta > 0) {
        slot_first = pg_list[0].y >> 8;
        n_local = (pg_list[n_cta - 1].y >> 8) - slot_first + 1;
    }
    for (int idx = threadIdx.x; idx < n_local * kMaxRep; idx += kThreads) cslot[idx] = 0.f;
    __syncthreads();                                                         // every stage consumed: the ring is free
    if (*abort_flag) return;

    // ---- merge the warps: reference maximum, sum, output, slot log-sums of the CTA ----
    // [warp][kMaxRep][D + 8]: with rows D floats apart the eight rows a warp stores together would share their banks
    constexpr int kORow = D + 8;
    static_assert(kWarps * kMaxRep * kORow * 4 <= C::kRingBytes, "the warps' outputs fit the idle ring");
    float *obuf = reinterpret_cast<float *>(smem);
    if (g < rep) {
#pragma unroll
        for (int nb = 0; nb < kNB; ++nb)
            *reinterpret_cast<float2 *>(obuf + (warp * kMaxRep + g) * kORow + nb * 8 + 2 * tq) = make_float2(o[nb][0], o[nb][1]);
    }
    if (warp < rep) {                                                        // warp h takes head h: lane w holds warp w's (m, l)
        const int h = warp;
        const float mw = lane < kWarps ? wm[lane * kMaxRep + h] : kNegInf;
        float M = mw;
#pragma unroll
        for (int of = 16; of > 0; of >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, of));
        const float f = (mw == kNegInf) ? 0.f : ex2(mw - M);
        float Lh = lane < kWarps ? wl[lane * kMaxRep + h] * f : 0.f;
#pragma unroll
        for (int of = 16; of > 0; of >>= 1) Lh += __shfl_xor_sync(0xffffffffu, Lh, of);
        if (lane < kWarps) weights[h * kMaxSplits + lane] = f;               // warp weights, reused below
        if (lane == 0) {
            cm[h] = (Lh > 0.f) ? M + lg2(Lh) : kNegInf;                      // log2-sum-exp of the CTA's range
            cl[h] = (Lh > 0.f) ? rcp(Lh) : 0.f;
        }
    }
    __syncthreads();
    // parked sums -> one log2-sum per (slot, head).  The reference is the log2-sum-exp of the CTA's whole range: no
    // slot's sum exceeds it, so the shares exp2(value - reference) are at most 1 and add up without a maximum pass
    // (a share below 2^-126 counts as nothing).
    const int n_ent = ctrs[1];
    for (int idx = threadIdx.x; idx < n_ent * rep; idx += kThreads) {
        const int e = idx / rep, h = idx % rep;
        const float v = ent_val[e * kMaxRep + h];
        if (v != kNegInf) atomicAdd(&cslot[(ent_slot[e] - slot_first) * kMaxRep + h], ex2(v - cm[h]));
    }
    // (the barrier that ends this pass comes after the output merge below, which does not depend on it)

    const bool single = p.n_splits == 1;
    const long long row_h0 = static_cast<long long>(ep.q_off) * p.Hq + it.kvh * rep;          // + h: (row, head) index
    const long long rh0 = static_cast<long long>(it.split) * p.n_q_total * p.Hq + row_h0;     // + h: partial index
    const int n_f4 = rep * D / 4;                                             // the rep output rows as float4
    for (int ff = threadIdx.x; ff < n_f4; ff += kThreads) {
        const int h = ff / (D / 4);
        float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
        float4 v[kWarps];
#pragma unroll
        for (int w = 0; w < kWarps; ++w)
            v[w] = *reinterpret_cast<const float4 *>(obuf + (w * kMaxRep + h) * kORow + (ff % (D / 4)) * 4);
#pragma unroll
        for (int w = 0; w < kWarps; ++w) {
            const float f = weights[h * kMaxSplits + w];
            a.x += f * v[w].x; a.y += f * v[w].y; a.z += f * v[w].z; a.w += f * v[w].w;
        }
        const float inv = cl[h];
        a.x *= inv; a.y *= inv; a.z *= inv; a.w *= inv;
        if (single) {
            uint2 o2;
            o2.x = pack_bf16(a.x, a.y);
            o2.y = pack_bf16(a.z, a.w);
            *reinterpret_cast<uint2 *>(static_cast<__nv_bfloat16 *>(p.out) + row_h0 * D + ff * 4) = o2;
        } else {
            *reinterpret_cast<float4 *>(p.part_o + rh0 * D + ff * 4) = a;
        }
    }
    if (!single) {
        if (threadIdx.x < rep) p.part_lse[rh0 + threadIdx.x] = cm[threadIdx.x];
        if (threadIdx.x == 0)
            p.part_rng[(it.split * static_cast<int>(gridDim.z) + it.ep) * p.Hkv + it.kvh] = make_int2(slot_first, n_local);
    }
    __syncthreads();                                                         // every share has been added
    if (single) {
        // the CTA saw the whole stream: a slot's share of the range is its mass
        if (p.mass)
            for (int idx = threadIdx.x; idx < rep * (G + 1); idx += kThreads) {
                const int h = idx / (G + 1), s = idx % (G + 1);
                const bool mine = s >= slot_first && s < slot_first + n_local;
                p.mass[(row_h0 + h) * p.mass_stride + s] = mine ? cslot[(s - slot_first) * kMaxRep + h] : 0.f;
            }
        return;
    }
    if (p.part_slot)                                                         // only the slots this range touched, as log2-sums
        for (int idx = threadIdx.x; idx < rep * n_local; idx += kThreads) {
            const int h = idx / n_local, sl = idx % n_local;
            const float sum = cslot[sl * kMaxRep + h];
            p.part_slot[(rh0 + h) * p.slot_stride + slot_first + sl] = (sum > 0.f) ? cm[h] + lg2(sum) : kNegInf;
        }

    // ---- the last CTA of this (episode, kv head) merges the splits ----
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        int *ctr = p.counters + it.ep * p.Hkv + it.kvh;
        const int prev = atomicAdd(ctr, 1);
        if (prev == p.n_splits - 1) {
            flags[1] = 1;
            *ctr = 0;                                                        // ready for the next launch
        }
    }
    __syncthreads();
    if (!flags[1]) return;
    __threadfence();
    const long long split_stride = static_cast<long long>(p.n_q_total) * p.Hq;
    // Round trip 1, everything that does not depend on anything else: the first partial outputs of every
    // thread, the splits' slot ranges (lane j of warp w keeps split w + j * kWarps) and the log-sum-exps.
    constexpr int kBatch = 8;
    const int groups = max(1, kThreads / n_f4);
    const int grp = threadIdx.x / n_f4, f = threadIdx.x % n_f4;
    const bool active = grp < groups;                                        // n_f4 <= kThreads for rep <= 8, D <= 128
    const float4 *po4 = reinterpret_cast<const float4 *>(p.part_o + row_h0 * D) + f;
    const long long po_stride4 = split_stride * D / 4;
    float4 pv[kBatch];
#pragma unroll
    for (int j = 0; j < kBatch; ++j) {
        const int k = grp + j * groups;
        pv[j] = (active && k < p.n_splits) ? __ldcg(po4 + k * po_stride4) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    // slot range of split k = warp + lane * kWarps (worked out from the plan at the start of the kernel)
    int2 my_rng = make_int2(0, 0);
    {
        const int k = warp + lane * kWarps;
        if (k < p.n_splits) my_rng = rng_tab[k];
    }
    // ... and the slot log-sums: the first 32 (head, slot) pairs of the splits warp and warp + kWarps
    float xs[2] = {kNegInf, kNegInf};
    if (p.mass) {
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const int k = warp + j * kWarps;
            const int first = __shfl_sync(0xffffffffu, my_rng.x, j), cnt = __shfl_sync(0xffffffffu, my_rng.y, j);
            if (k < p.n_splits && lane < cnt * rep)
                xs[j] = __ldcg(p.part_slot + (k * split_stride + row_h0 + lane / cnt) * p.slot_stride + first + lane % cnt);
        }
    }
    for (int h = warp; h < rep; h += kWarps) {                               // weights of the splits: one warp per head
        const float my0 = lane < p.n_splits ? __ldcg(p.part_lse + lane * split_stride + row_h0 + h) : kNegInf;
        const float my1 = lane + 32 < p.n_splits ? __ldcg(p.part_lse + (lane + 32) * split_stride + row_h0 + h) : kNegInf;
        float mxv = fmaxf(my0, my1);
#pragma unroll
        for (int of = 16; of > 0; of >>= 1) mxv = fmaxf(mxv, __shfl_xor_sync(0xffffffffu, mxv, of));
        float sum = (my0 != kNegInf ? ex2(my0 - mxv) : 0.f) + (my1 != kNegInf ? ex2(my1 - mxv) : 0.f);
#pragma unroll
        for (int of = 16; of > 0; of >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, of);
        const float lse = (mxv != kNegInf) ? mxv + lg2(sum) : kNegInf;
        weights[h * kMaxSplits + lane] = (my0 != kNegInf) ? ex2(my0 - lse) : 0.f;
        if (lane + 32 < kMaxSplits) weights[h * kMaxSplits + lane + 32] = (my1 != kNegInf) ? ex2(my1 - lse) : 0.f;
        if (lane == 0) cm[h] = lse;
    }
    // per-slot table in the idle ring (behind the reduction buffer), zeroed before the barrier
    constexpr int kRedFloats = kThreads * 4;
    float *red = reinterpret_cast<float *>(smem);                            // [group][rep * D] partial outputs
    float *tab = red + kRedFloats;                                           // [rep][G + 1]
    constexpr int kTabCap = (C::kRingBytes - kRedFloats * 4) / 4;
    const bool tab_fits = rep * (G + 1) <= kTabCap;
    if (p.mass && tab_fits)
        for (int idx = threadIdx.x; idx < rep * (G + 1); idx += kThreads) tab[idx] = 0.f;
    __syncthreads();

    // the slot log-sums of every split (only the slots its range touched): what was fetched above, then the rest
    if (p.mass && tab_fits) {
        for (int j = 0; warp + j * kWarps < p.n_splits; ++j) {
            const int k = warp + j * kWarps;
            const int first = __shfl_sync(0xffffffffu, my_rng.x, j), cnt = __shfl_sync(0xffffffffu, my_rng.y, j);
            for (int idx = lane; idx < cnt * rep; idx += 32) {
                const int h = idx / cnt, sl = idx % cnt;
                const float lse = cm[h];
                const float x = (j < 2 && idx < 32) ? (j == 0 ? xs[0] : xs[1])
                                                    : __ldcg(p.part_slot + (k * split_stride + row_h0 + h) * p.slot_stride + first + sl);
                if (lse != kNegInf && x != kNegInf) atomicAdd(&tab[h * (G + 1) + first + sl], ex2(x - lse));
            }
        }
    }
    // output: float4 f of split k goes to thread (k mod groups, f)
    if (active) {
        const int h = f / (D / 4);
        float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int j = 0; j < kBatch; ++j) {
            const int k = grp + j * groups;
            const float w = (k < p.n_splits) ? weights[h * kMaxSplits + k] : 0.f;
            a.x += w * pv[j].x; a.y += w * pv[j].y; a.z += w * pv[j].z; a.w += w * pv[j].w;
        }
#pragma unroll 1
        for (int k = grp + kBatch * groups; k < p.n_splits; k += groups) {   // more splits than one batch covers
            const float w = weights[h * kMaxSplits + k];
            const float4 v = __ldcg(po4 + k * po_stride4);
            a.x += w * v.x; a.y += w * v.y; a.z += w * v.z; a.w += w * v.w;
        }
        *reinterpret_cast<float4 *>(red + (grp * n_f4 + f) * 4) = a;
    }
    __syncthreads();
    if (threadIdx.x < n_f4) {
        float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 1
        for (int gi = 0; gi < groups; ++gi) {
            const float4 v = *reinterpret_cast<const float4 *>(red + (gi * n_f4 + f) * 4);
            t.x += v.x; t.y += v.y; t.z += v.z; t.w += v.w;
        }
        uint2 o2;
        o2.x = pack_bf16(t.x, t.y);
        o2.y = pack_bf16(t.z, t.w);
        *reinterpret_cast<uint2 *>(static_cast<__nv_bfloat16 *>(p.out) + row_h0 * D + f * 4) = o2;
    }
    if (!p.mass) return;
    if (tab_fits) {
        for (int idx = threadIdx.x; idx < rep * (G + 1); idx += kThreads) {
            const int h = idx / (G + 1), sidx = idx % (G + 1);
            p.mass[(row_h0 + h) * p.mass_stride + sidx] = tab[idx];
        }
    } else {
        // more slots than the table holds: one thread per (head, slot), splits in order
        for (int idx = threadIdx.x; idx < rep * (G + 1); idx += kThreads) {
            const int h = idx / (G + 1), sidx = idx % (G + 1);
            const float lse = cm[h];
            float v = 0.f;
#pragma unroll 1
            for (int k = 0; k < p.n_splits; ++k) {
                const int2 rng = __ldcg(p.part_rng + (k * static_cast<int>(gridDim.z) + it.ep) * p.Hkv + it.kvh);
                if (sidx < rng.x || sidx >= rng.x + rng.y) continue;
                const float x = __ldcg(p.part_slot + (k * split_stride + row_h0 + h) * p.slot_stride + sidx);
                if (lse != kNegInf && x != kNegInf) v += ex2(x - lse);
            }
            p.mass[(row_h0 + h) * p.mass_stride + sidx] = v;
        }
    }
}

}  // namespace

size_t decode_smem_bytes(int head_dim)
{
    return head_dim == 128 ? DecCfg<128>::kSmemBytes : DecCfg<64>::kSmemBytes;
}

cudaError_t prepare_decode(int head_dim)
{
    if (head_dim == 128)
        return cudaFuncSetAttribute(decode_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, DecCfg<128>::kSmemBytes);
    if (head_dim == 64)
        return cudaFuncSetAttribute(decode_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, DecCfg<64>::kSmemBytes);
    return cudaErrorInvalidValue;
}

cudaError_t launch_decode(const DecodeParams &p, int head_dim, int batch, cudaStream_t st)
{
    if (batch <= 0 || p.n_splits <= 0) return cudaSuccess;
    const dim3 grid(p.n_splits, p.Hkv, batch);
    cudaError_t e;
    if (head_dim == 128)
        e = launch_pdl(decode_kernel<128>, grid, dim3(kThreads), DecCfg<128>::kSmemBytes, st, p);
    else if (head_dim == 64)
        e = launch_pdl(decode_kernel<64>, grid, dim3(kThreads), DecCfg<64>::kSmemBytes, st, p);
    else
        return cudaErrorInvalidValue;
    return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace enl
