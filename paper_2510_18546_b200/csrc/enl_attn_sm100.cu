// Selective-KV flash attention with fused per-group mass, sm_100a (tcgen05 + TMEM + TMA).
//
// What it computes (paper, App. A: softmax(Q K^T / sqrt(D)) V; App. C: the prompt is the selected
// groups followed by the new tokens; Sec. 3.3: attention between new tokens and a group):
// one CTA takes two Q tiles of 128 rows each -- (128/rep) consecutive query tokens x the rep q heads
// that read one kv head -- and walks the key stream of its episode: the selected groups' pages in
// list order (eight 16-token pages per 128-key tile, fetched as separate TMA boxes from wherever the
// pages lie in the pool), then the new-token keys up to the causal limit.  Per tile:
//   S_i = Q_i K^T            tcgen05.mma, operands in shared memory, accumulator in TMEM
//   p   = exp2(S * c - m)    one thread per row, fp32; padding and causally hidden columns -> 0
//   O_i += P_i V             tcgen05.mma, P (bf16) read from TMEM, V from shared memory
// The row sum of p is split by the slot (selected group, or the new tokens) each 16-key page belongs
// to; when a slot ends its log2-sum-exp is parked (in shared memory for calls with few slots, else in
// the mass buffer), and after the last tile the parked values are turned into probabilities.  With KV splits every split writes partial results that a
// second kernel merges, or (two splits, head_dim 128) the two CTAs of a cluster merge in place.
//
// Roles (12 warps): warps 0-3 are the softmax warpgroup of Q tile 0, warps 4-7 that of Q tile 1: one
// thread per query row holds the row's 128 scores of a tile in registers, so the row maximum, the
// exponentials and the eight page sums need no exchange between threads.  Warp 8 is the TMA producer,
// warp 9 the MMA issuer (and TMEM owner), warps 10-11 idle: they complete the third warpgroup so that
// setmaxnreg can move its registers to the softmax warpgroups.
// The two Q tiles alternate on the tensor pipe: while one tile's softmax runs, the pipe does the other
// tile's P V and the next Q K^T.  P is handed over in two halves of 64 keys so that P V starts while
// the second half's exponentials are still being taken; everything that is not needed for P (row and
// page sums, slot book-keeping) is done after the hand-over, under the MMAs.
// TMEM columns: S0 [0,128) S1 [128,256) O0 [256,384) O1 [384,512); P_i (bf16 pairs) overwrites columns
// [0,64) of S_i once the row's scores are in registers.
#include <cuda_bf16.h>

#include "enl_internal.h"
#include "tmem_ops.cuh"

namespace enl {
namespace {

constexpr int kThreads      = 384;
constexpr int kSoftmaxWarps = 8;
constexpr int kRegsSoftmax  = 208;            // 256 x 208 + 128 x 80 <= 384 x 168, what the launch allocates
constexpr int kRegsOther    = 80;
constexpr int kProducerWarp = 8;
constexpr int kMmaWarp      = 9;
constexpr uint32_t kTmemCols = 512;
constexpr int kParkSlots = 28;                // calls with up to this many mass slots park their slot sums in shared memory
constexpr float kRescaleThreshold = 8.0f;     // log2 units: p stays below 2^8 between updates of the reference
constexpr unsigned long long kWaitLimitNs = 1000ull * 1000ull * 1000ull;
constexpr uint32_t kFull = 0xffffffffu;

template <int D>
struct Cfg {
    static constexpr int kHalves    = D / 64;             // 64-channel (128-byte) column blocks
    static constexpr int kHalfBytes = 128 * 128;          // 128 rows x 128 B
    static constexpr int kTileBytes = kHalves * kHalfBytes;
    static constexpr int kStages    = (D == 128) ? 4 : 8;
    static constexpr int kBarOff    = (kQTiles + kStages) * kTileBytes;
    // pair merge: what the other CTA of the cluster knows about this CTA's rows, [tile][128] x (m, l, shared-slot log-sum, -)
    static constexpr int kXpeerOff  = kBarOff + 512;
    // slot log-sums of calls with at most kParkSlots slots, [tile][slot][128 rows] fp32 (what is left of the 227 KB)
    static constexpr int kParkOff   = kXpeerOff + kQTiles * 128 * 16;
    static constexpr int kSmemBytes = kParkOff + kQTiles * kParkSlots * 128 * 4 + 1024;   // + alignment slack
};

// ---- small PTX wrappers ------------------------------------------------------------------
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
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
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
// A test that never suspends (about 35 cycles until its result can be used, half of a poll with a suspend hint).
__device__ __forceinline__ bool mbar_test(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// The same poll with acquire semantics at cluster scope: data another CTA of the cluster wrote before its
// release.cluster arrival is visible afterwards.  No suspend hint: a thread suspended with the long hint was seen
// to sleep through an arrival that came from the other CTA.
__device__ __forceinline__ bool mbar_try_wait_cluster(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Distributed shared memory of a two-CTA cluster: address of the peer's copy of a local shared-memory location,
// stores to it, and arrivals on its barriers.
__device__ __forceinline__ uint32_t cluster_rank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t peer_addr(uint32_t local, uint32_t rank)
{
    uint32_t a;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(a) : "r"(local), "r"(rank));
    return a;
}
// 16-byte store into the peer's shared memory whose completion is counted (in bytes) on a barrier of the peer: the
// sender needs no release fence, which would also wait for its earlier global stores
__device__ __forceinline__ void peer_push4(uint32_t addr, float a, float b, float c, float d, uint32_t bar_peer)
{
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.f32 [%0], {%1, %2, %3, %4}, [%5];"
                 ::"r"(addr), "f"(a), "f"(b), "f"(c), "f"(d), "r"(bar_peer) : "memory");
}
// an arrival that publishes nothing (a plain "go ahead")
__device__ __forceinline__ void peer_arrive_relaxed(uint32_t bar)
{
    asm volatile("mbarrier.arrive.relaxed.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void peer_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar) : "memory");
}
// bulk copy from this CTA's shared memory into the peer's; the bytes are counted on a barrier of the peer
__device__ __forceinline__ void peer_bulk_copy(uint32_t dst_peer, uint32_t src_local, uint32_t bytes, uint32_t bar_peer)
{
    asm volatile("cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst_peer), "r"(src_local), "r"(bytes), "r"(bar_peer) : "memory");
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ unsigned long long global_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait: gives up about kWaitLimitNs after its 16th failed poll, or when another role has raised the abort flag.
// The result is made warp-uniform so that warp-collective tcgen05 instructions stay converged.
template <bool kCluster = false>
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag,
                                          int32_t *status)
{
    auto poll = [&]() { return kCluster ? mbar_try_wait_cluster(bar, parity) : mbar_try_wait(bar, parity); };
    bool ok = kCluster ? poll() : mbar_test(bar, parity);       // the common case: already complete
    if (!ok) {
        // the clock is read only every 16 failed polls (the first reading starts the limit): a poll already
        // sleeps inside the instruction
        unsigned long long t0 = 0;
        uint32_t spins = 0;
        while (!(ok = poll())) {
            if ((++spins & 15u) == 0u) {
                if (*abort_flag) break;
                const unsigned long long now = global_ns();
                if (t0 == 0) {
                    t0 = now;
                } else if (now - t0 > kWaitLimitNs) {
                    *abort_flag = 1;
                    atomicExch(status, 1);
                    break;
                }
            }
        }
    }
    return __all_sync(kFull, ok);
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *tm, int x, int y, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(tm), "r"(x), "r"(y), "r"(bar) : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *tm, int x, int y, int z, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(tm), "r"(x), "r"(y), "r"(z), "r"(bar) : "memory");
}
// Bring a box into the L2 without a destination in the SM: nothing is observed, so these may run before the wait for
// the previous kernel of the stream (the L2 is the point of coherence: a later write to those lines updates them).
__device__ __forceinline__ void tma_prefetch_2d(const CUtensorMap *tm, int x, int y)
{
    asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global.tile [%0, {%1, %2}];" ::"l"(tm), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void tma_prefetch_3d(const CUtensorMap *tm, int x, int y, int z)
{
    asm volatile("cp.async.bulk.prefetch.tensor.3d.L2.global.tile [%0, {%1, %2, %3}];"
                 ::"l"(tm), "r"(x), "r"(y), "r"(z) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after()  { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// D[tmem] (+)= A[smem] * B[smem] and D[tmem] (+)= A[tmem] * B[smem].  The whole warp executes the surrounding code
// and these wrappers; only the lane with `issue` != 0 issues the instruction.  Issuing from inside a one-lane branch
// was measured at ~60 cycles per MMA (a diverged warp pays the full latency of every instruction and cannot use the
// uniform datapath for the descriptors), against ~10 cycles this way; the pipe retires an MMA every ~65 cycles.
// The shared-memory descriptors are given as (low word, high word): the high word is constant and the low word (the
// start address field) moves by a small constant from one MMA to the next.
__device__ __forceinline__ void mma_ss2(uint32_t d, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi,
                                        uint32_t idesc, uint32_t acc, uint32_t issue)
{
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t.reg .b64 da, db;\n\t"
        "mov.b64 da, {%1, %2};\n\tmov.b64 db, {%3, %4};\n\tsetp.ne.b32 p, %6, 0;\n\tsetp.ne.b32 q, %7, 0;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, p;\n\t}"
        ::"r"(d), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(acc), "r"(issue) : "memory");
}
__device__ __forceinline__ void mma_ts2(uint32_t d, uint32_t a, uint32_t b_lo, uint32_t b_hi, uint32_t idesc, uint32_t acc,
                                        uint32_t issue)
{
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t.reg .b64 db;\n\t"
        "mov.b64 db, {%2, %3};\n\tsetp.ne.b32 p, %5, 0;\n\tsetp.ne.b32 q, %6, 0;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %4, p;\n\t}"
        ::"r"(d), "r"(a), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(acc), "r"(issue) : "memory");
}
__device__ __forceinline__ void tc_commit_if(uint32_t bar, uint32_t issue)
{
    asm volatile(
        "{\n\t.reg .pred q;\n\tsetp.ne.b32 q, %1, 0;\n\t"
        "@q tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}"
        ::"r"(bar), "r"(issue) : "memory");
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

// 3-input max and packed 2 x fp32 arithmetic (one issue slot for two lanes of work)
__device__ __forceinline__ float fmax3(float a, float b, float c)
{
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ uint64_t pack2(float lo, float hi)
{
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float &lo, float &hi)
{
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c)
{
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b)
{
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint32_t bf16x2(float lo, float hi)
{
    const __nv_bfloat162 b = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t *>(&b);
}

// Shared-memory matrix descriptor, 128-byte swizzle, rows of 128 B, 8-row groups 1024 B apart.
// K-major operand (the contraction dimension is contiguous): LBO unused.
// MN-major operand: LBO = distance between 64-element column blocks.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes)
{
    uint64_t d = 0;
    d |= static_cast<uint64_t>((addr & 0x3FFFFu) >> 4);               // start address
    d |= static_cast<uint64_t>((lbo_bytes >> 4) & 0x3FFFu) << 16;      // leading byte offset
    d |= static_cast<uint64_t>(1024u >> 4) << 32;                      // stride byte offset
    d |= static_cast<uint64_t>(1) << 46;                               // descriptor version (sm_100)
    d |= static_cast<uint64_t>(2) << 61;                               // 128-byte swizzle
    return d;
}
// Instruction descriptor, kind::f16: bf16 x bf16 -> fp32, M = 128.
__host__ __device__ constexpr uint32_t make_idesc(int n, bool b_mn_major)
{
    return (1u << 4)                              // D format fp32
         | (1u << 7) | (1u << 10)                 // A, B format bf16
         | ((b_mn_major ? 1u : 0u) << 16)         // B major
         | (static_cast<uint32_t>(n >> 3) << 17)  // N
         | (static_cast<uint32_t>(128 >> 4) << 24);  // M
}

constexpr float kNegInf = -__builtin_huge_valf();

// ---- the kernel ----------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(kThreads, 1) attn_kernel(const __grid_constant__ AttnParams p)
{
    using C = Cfg<D>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t sbase = (raw + 1023u) & ~1023u;               // 1024-B aligned (swizzle atoms)
    uint8_t *smem = smem_raw + (sbase - raw);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // shared-memory map
    auto q_addr     = [&](int i) { return sbase + static_cast<uint32_t>(i * C::kTileBytes); };
    auto stage_addr = [&](int s) { return sbase + static_cast<uint32_t>((kQTiles + s) * C::kTileBytes); };
    const uint32_t bar0 = sbase + C::kBarOff;
    const uint32_t bar_q_full = bar0;
    auto bar_kv_full  = [&](int s) { return bar0 + 8u * (1 + s); };
    auto bar_kv_empty = [&](int s) { return bar0 + 8u * (1 + C::kStages + s); };
    auto bar_s_full   = [&](int i) { return bar0 + 8u * (1 + 2 * C::kStages + i); };
    auto bar_p_half   = [&](int i, int hf) { return bar0 + 8u * (3 + 2 * C::kStages + 2 * i + hf); };   // keys 0..63 / 64..127 of P_i
    auto bar_o_done   = [&](int i) { return bar0 + 8u * (7 + 2 * C::kStages + i); };
    // pair merge (cluster of two): the peer's row sums have arrived / the peer's partial output has arrived /
    // the peer's K/V ring is idle and may be written / the peer has received what this CTA staged for it
    const uint32_t bar_peer_ml = bar0 + 8u * (9 + 2 * C::kStages);
    const uint32_t bar_peer_o = bar0 + 8u * (10 + 2 * C::kStages);
    const uint32_t bar_peer_free = bar0 + 8u * (11 + 2 * C::kStages);
    const uint32_t bar_peer_ack = bar0 + 8u * (12 + 2 * C::kStages);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + C::kBarOff + 8 * (13 + 2 * C::kStages));
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    // work item
    const Item it = p.items[blockIdx.x];
    const EpInfo ep = p.eps[it.ep];
    const int rep = p.rep;
    const int tile_tokens = kTileRows / rep;
    const int t_hi = min(it.t0 + kQTiles * tile_tokens, ep.n_q);        // exclusive
    const int n_qt = (t_hi - it.t0 > tile_tokens) ? 2 : 1;
    const int c_max = ep.n_new - ep.n_q + t_hi - 1;                      // last new key any row sees
    const int n_new_tiles = c_max / kTileKeys + 1;
    const int total_tiles = ep.n_ctiles + n_new_tiles;
    const int j_beg = static_cast<int>(static_cast<long long>(total_tiles) * it.split / p.n_splits);
    const int j_end = static_cast<int>(static_cast<long long>(total_tiles) * (it.split + 1) / p.n_splits);
    const int n_tiles = j_end - j_beg;

    // ---- set-up ----
    if (threadIdx.x == 0) {
        *abort_flag = 0;
        mbar_init(bar_q_full, 1);
        for (int s = 0; s < C::kStages; ++s) { mbar_init(bar_kv_full(s), 1); mbar_init(bar_kv_empty(s), 1); }
        for (int i = 0; i < kQTiles; ++i) {
            mbar_init(bar_s_full(i), 1);
            mbar_init(bar_p_half(i, 0), 4);       // one arrival per softmax warp of the tile
            mbar_init(bar_p_half(i, 1), 4);
            mbar_init(bar_o_done(i), 1);
        }
        mbar_init(bar_peer_ml, 1);                                   // this thread's arrival below + 16 bytes per row from the peer
        mbar_init(bar_peer_o, 1);                                    // this thread's arrival below + 64 KB from the peer
        mbar_init(bar_peer_free, 1);
        mbar_init(bar_peer_ack, 1);
        if (p.pair_merge) {
            mbar_expect_tx(bar_peer_ml, static_cast<uint32_t>(n_qt * 128 * 16));
            mbar_expect_tx(bar_peer_o, 4u * 16384u);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == kMmaWarp) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_slot)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const bool pair = p.pair_merge != 0;
    if (pair) cluster_sync_all();                // the peer's barriers exist before anything is sent to them
    // everything above touched only shared memory, TMEM and the gather plan; from here on the caller's tensors,
    // the pool and the scratch are read and written, so the previous kernel of the stream must have finished
    pdl_trigger();
    // While the previous kernel drains, ask what the first S tile needs into the L2: the Q tiles and the first two
    // key tiles' K and V (cached pages; new-token tiles only when the stream starts with them).
    // (Only CTAs of the first wave wait for the previous kernel; for the others this would be loads issued twice.)
    if (warp == kProducerWarp && n_tiles > 0 && static_cast<int>(blockIdx.x) < p.first_wave) {
        if (lane < n_qt * C::kHalves)
            tma_prefetch_3d(&p.tm_q, (lane % C::kHalves) * 64, it.kvh * rep, ep.q_off + it.t0 + (lane / C::kHalves) * tile_tokens);
        for (int j = j_beg; j < min(j_beg + 2, j_end); ++j) {
            if (j < ep.n_ctiles) {
                if (lane < kPagesPerTile) {
                    const int row = (p.stream_page[ep.stream_off + j * kPagesPerTile + lane] * p.Hkv + it.kvh) * kPageTokens;
                    for (int hf = 0; hf < C::kHalves; ++hf) {
                        tma_prefetch_2d(&p.tm_kpool, hf * 64, row);
                        tma_prefetch_2d(&p.tm_vpool, hf * 64, row);
                    }
                }
            } else if (lane < 2 * C::kHalves) {
                tma_prefetch_3d(lane < C::kHalves ? &p.tm_knew : &p.tm_vnew, (lane % C::kHalves) * 64, it.kvh,
                                ep.new_off + (j - ep.n_ctiles) * kTileKeys);
            }
        }
    }
    pdl_wait();

    bool ok = true;

    if (warp >= kSoftmaxWarps) {
      asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsOther));
      if (warp == kProducerWarp) {
        // ================= TMA producer =================
        if (n_tiles > 0) {
            if (lane == 0) {
                mbar_expect_tx(bar_q_full, static_cast<uint32_t>(n_qt * C::kTileBytes));
                for (int i = 0; i < n_qt; ++i)
                    for (int hf = 0; hf < C::kHalves; ++hf)
                        tma_load_3d(q_addr(i) + hf * C::kHalfBytes, &p.tm_q, hf * 64, it.kvh * rep,
                                    ep.q_off + it.t0 + i * tile_tokens, bar_q_full);
            }
            int fill = 0;
            for (int j = j_beg; j < j_end && ok; ++j) {
                const bool cached = j < ep.n_ctiles;
                int page = 0;
                if (cached && lane < kPagesPerTile)
                    page = p.stream_page[ep.stream_off + j * kPagesPerTile + lane];
                for (int kv = 0; kv < 2; ++kv, ++fill) {
                    const int st = fill % C::kStages;
                    if (fill >= C::kStages) {
                        ok = mbar_wait(bar_kv_empty(st), static_cast<uint32_t>((fill / C::kStages - 1) & 1),
                                       abort_flag, p.status);
                        if (!ok) break;
                    }
                    const uint32_t full = bar_kv_full(st);
                    if (lane == 0) mbar_expect_tx(full, static_cast<uint32_t>(C::kTileBytes));
                    __syncwarp();
                    const uint32_t dst = stage_addr(st);
                    if (cached) {
                        if (lane < kPagesPerTile) {
                            const CUtensorMap *tm = kv ? &p.tm_vpool : &p.tm_kpool;
                            const int row = (page * p.Hkv + it.kvh) * kPageTokens;
                            for (int hf = 0; hf < C::kHalves; ++hf)
                                tma_load_2d(dst + hf * C::kHalfBytes + lane * (kPageTokens * 128), tm,
                                            hf * 64, row, full);
                        }
                    } else if (lane == 0) {
                        const CUtensorMap *tm = kv ? &p.tm_vnew : &p.tm_knew;
                        const int krow = ep.new_off + (j - ep.n_ctiles) * kTileKeys;
                        for (int hf = 0; hf < C::kHalves; ++hf)
                            tma_load_3d(dst + hf * C::kHalfBytes, tm, hf * 64, it.kvh, krow, full);
                    }
                }
            }
            // error path only: let the copies already in flight land before the CTA retires
            if (!ok) {
                const int first = fill > C::kStages ? fill - C::kStages : 0;
                for (int f = first; f < fill; ++f) {
                    const unsigned long long t0 = global_ns();
                    while (!mbar_try_wait(bar_kv_full(f % C::kStages), static_cast<uint32_t>((f / C::kStages) & 1)) &&
                           global_ns() - t0 < 2000000ull) { }
                }
            }
        }
      } else if (warp == kMmaWarp) {
        // ================= MMA issuer =================
        if (n_tiles > 0) {
            constexpr uint32_t idesc_qk = make_idesc(kTileKeys, false);
            constexpr uint32_t idesc_pv = make_idesc(D, true);
            auto tmem_s = [&](int i) { return tmem_base + static_cast<uint32_t>(i * 128); };
            auto tmem_o = [&](int i) { return tmem_base + static_cast<uint32_t>(256 + i * 128); };
            // descriptor words: Q tile i and ring stage st start (kTileBytes >> 4) address units apart
            const uint64_t dq0 = smem_desc(q_addr(0), 16), dk0 = smem_desc(stage_addr(0), 16),
                           dv0 = smem_desc(stage_addr(0), C::kHalfBytes);
            const uint32_t dq_lo = static_cast<uint32_t>(dq0), dq_hi = static_cast<uint32_t>(dq0 >> 32);
            const uint32_t dk_lo = static_cast<uint32_t>(dk0), dk_hi = static_cast<uint32_t>(dk0 >> 32);
            const uint32_t dv_lo = static_cast<uint32_t>(dv0), dv_hi = static_cast<uint32_t>(dv0 >> 32);
            constexpr uint32_t kTileUnits = C::kTileBytes >> 4;
            const uint32_t issue = lane == 0 ? 1u : 0u;
            auto issue_qk = [&](int i, int st) {
                const uint32_t a = dq_lo + static_cast<uint32_t>(i) * kTileUnits, b = dk_lo + static_cast<uint32_t>(st) * kTileUnits;
                const uint32_t d = tmem_s(i);
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    constexpr uint32_t kHalfUnits = C::kHalfBytes >> 4;
                    const uint32_t off = static_cast<uint32_t>((kk >> 2) * kHalfUnits + (kk & 3) * 2);   // 32 bytes per 16 channels
                    mma_ss2(d, a + off, dq_hi, b + off, dk_hi, idesc_qk, kk > 0 ? 1u : 0u, issue);
                }
                tc_commit_if(bar_s_full(i), issue);
            };
            // O_i (+)= P_i[:, 64 hf .. 64 hf + 63] V[64 hf .. 64 hf + 63, :]; P of keys 2c, 2c+1 sits in column c of S_i
            auto issue_pv = [&](int i, int st, int hf, bool first_tile) {
                const uint32_t b = dv_lo + static_cast<uint32_t>(st) * kTileUnits + static_cast<uint32_t>(hf) * (4u * 128u);
                const uint32_t d = tmem_o(i), a = tmem_s(i) + static_cast<uint32_t>(hf * 32);
#pragma unroll
                for (int k4 = 0; k4 < 4; ++k4)                          // 16 keys = 16 rows of 128 B = 128 address units, 8 columns of P
                    mma_ts2(d, a + static_cast<uint32_t>(k4 * 8), b + static_cast<uint32_t>(k4 * 128), dv_hi, idesc_pv,
                            (first_tile && hf == 0 && k4 == 0) ? 0u : 1u, issue);
            };
            auto commit_to = [&](uint32_t bar) { tc_commit_if(bar, issue); };
            auto wait_full = [&](int f) {
                return mbar_wait(bar_kv_full(f % C::kStages), static_cast<uint32_t>((f / C::kStages) & 1),
                                 abort_flag, p.status);
            };

            // A barrier the issuer will need is tested one batch of MMAs ahead ("armed"), so that the test's latency
            // passes while the batch is issued; only a barrier that was not complete then is waited for.  The queue in
            // front of the pipe holds about four MMAs: a wait of a few hundred cycles between two batches empties it.
            struct Pending { uint32_t bar, par; bool pre; };
            auto arm = [&](uint32_t bar, uint32_t par) { return Pending{bar, par, mbar_test(bar, par)}; };
            auto await = [&](const Pending &w) {
                return __all_sync(kFull, w.pre) ? true : mbar_wait(w.bar, w.par, abort_flag, p.status);
            };
            auto full_bar = [&](int f) { return bar_kv_full(f % C::kStages); };
            auto full_par = [&](int f) { return static_cast<uint32_t>((f / C::kStages) & 1); };

            ok = mbar_wait(bar_q_full, 0, abort_flag, p.status);
            if (ok) ok = wait_full(0);
            if (ok) {
                tc_fence_after();
                for (int i = 0; i < n_qt; ++i) issue_qk(i, 0);
                commit_to(bar_kv_empty(0));
            }
            Pending w_v = arm(full_bar(1), full_par(1));                // V of the first tile
            Pending w_p = arm(bar_p_half(0, 0), 0u);                    // first half of P_0
            for (int jj = 0; jj < n_tiles && ok; ++jj) {
                const int fv = 2 * jj + 1, fk = 2 * jj + 2;             // ring slots of V_jj and K_{jj+1}
                const bool more = jj + 1 < n_tiles;
                const uint32_t par = static_cast<uint32_t>(jj & 1);
                for (int i = 0; i < n_qt; ++i) {
                    const bool last_i = i == n_qt - 1;
                    if (i == 0) ok = await(w_v);
                    if (ok) ok = await(w_p);
                    if (!ok) break;
                    tc_fence_after();
                    const Pending w_h1 = arm(bar_p_half(i, 1), par);
                    issue_pv(i, fv % C::kStages, 0, jj == 0);
                    ok = await(w_h1);
                    if (!ok) break;
                    tc_fence_after();
                    Pending w_k = {0u, 0u, true};
                    if (more && i == 0) w_k = arm(full_bar(fk), full_par(fk));
                    if (!more && !last_i) w_p = arm(bar_p_half(i + 1, 0), par);
                    issue_pv(i, fv % C::kStages, 1, false);
                    if (last_i) commit_to(bar_kv_empty(fv % C::kStages));
                    if (!more) commit_to(bar_o_done(i));
                    if (more) {
                        ok = await(w_k);
                        if (!ok) break;
                        tc_fence_after();
                        // what follows Q_i K^T: the next tile's P of this key tile, or (after the last Q tile) V and P_0 of the next
                        if (!last_i) {
                            w_p = arm(bar_p_half(i + 1, 0), par);
                        } else {
                            w_v = arm(full_bar(fv + 2), full_par(fv + 2));
                            w_p = arm(bar_p_half(0, 0), par ^ 1u);
                        }
                        issue_qk(i, fk % C::kStages);
                        if (last_i) commit_to(bar_kv_empty(fk % C::kStages));
                    }
                }
            }
            // pair merge: once every MMA of this CTA has completed, its K/V ring is idle and the peer may write
            // into it (only a CTA that finishes a Q tile receives anything)
            if (ok && pair && it.split < n_qt) {
                for (int i = 0; i < n_qt && ok; ++i) ok = mbar_wait(bar_o_done(i), 0, abort_flag, p.status);
                if (ok && lane == 0) peer_arrive(peer_addr(bar_peer_free, cluster_rank() ^ 1u));
            }
        }
      }
    } else {
      asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegsSoftmax));
      if ((warp >> 2) < n_qt) {
        // ================= softmax / epilogue: one thread per query row =================
        const int i = warp >> 2;                                   // Q tile
        const int q4 = warp & 3;                                   // TMEM lane quadrant
        const int r = q4 * 32 + lane;
        const int t = it.t0 + i * tile_tokens + r / rep;           // episode-relative query token
        const int h = it.kvh * rep + r % rep;
        const bool row_valid = t < ep.n_q;
        const int c = min(ep.n_new - ep.n_q + t, ep.n_new - 1);    // last visible new key
        const int c_lo = ep.n_new - ep.n_q + it.t0 + i * tile_tokens;   // the same for the tile's first row: every row sees at least this far
        const int G = ep.n_slots;
        const uint32_t lane_sel = static_cast<uint32_t>(q4 * 32) << 16;
        const uint32_t t_s = tmem_base + lane_sel + static_cast<uint32_t>(i * 128);
        const uint32_t t_o = tmem_base + lane_sel + static_cast<uint32_t>(256 + i * 128);
        const bool split_mode = p.n_splits > 1 && !pair;
        const long long grow = static_cast<long long>(ep.q_off) + t;   // global query row
        const long long rh = (split_mode ? (static_cast<long long>(it.split) * p.n_q_total + grow) : grow) * p.Hq + h;
        // Where this row's slot log-sums are parked until the row's total is known: shared memory when the call has few
        // slots (one store per slot end, no round trip to the L2 at the end), else the buffer that takes the result.
        float *slot_out = nullptr;
        if (row_valid) {
            if (split_mode) { if (p.part_slot) slot_out = p.part_slot + rh * p.mass_stride; }
            else if (p.mass) slot_out = p.mass + rh * p.mass_stride;
        }
        const bool park_smem = G + 1 <= kParkSlots;
        float *park_row = reinterpret_cast<float *>(smem + C::kParkOff) + i * (kParkSlots * 128) + r;   // + slot * 128
        const float scale = p.scale_log2;

        // Pair merge: the slot in which the two splits meet is walked by both.  Split 0 writes it (adding what
        // split 1 sends); split 1 keeps its part in `bnd` instead of storing it.
        int shared_slot = -1, skip_slot = -1;
        float bnd = kNegInf;
        if (pair) {
            const int jb = (it.split == 0) ? j_end : j_beg;         // first tile of split 1
            const int last0 = (jb > ep.n_ctiles) ? G : (__ldg(p.stream_meta + ep.stream_off + jb * kPagesPerTile - 1) >> 8);
            const int first1 = (jb < ep.n_ctiles) ? (__ldg(p.stream_meta + ep.stream_off + jb * kPagesPerTile) >> 8) : G;
            if (last0 == first1) { shared_slot = last0; if (it.split == 1) skip_slot = last0; }
        }
        float m = kNegInf, l = 0.f, acc = 0.f;                     // reference (log2 units), row sum, sum of the current slot
        int cur_slot = -1;
        // the slot that ends parks its log2-sum-exp
        auto park = [&](float m_ref) {
            if (cur_slot >= 0) {
                const float v = lg2(acc) + m_ref;
                if (cur_slot == skip_slot) bnd = v;
                else if (park_smem) park_row[cur_slot * 128] = v;
                else if (slot_out) slot_out[cur_slot] = v;
            }
        };

        // Page words of a tile, one per lane 0..7 (slot << 8 | valid keys); a new-token tile is one slot (G).  They
        // are fetched one tile ahead: the load's latency would otherwise sit between two tiles of this warp.
        auto load_meta = [&](int j) -> int {
            int w = (G << 8) | kPageTokens;
            if (j < ep.n_ctiles && lane < kPagesPerTile) w = __ldg(p.stream_meta + ep.stream_off + j * kPagesPerTile + lane);
            return w;
        };
        int meta_next = n_tiles > 0 ? load_meta(j_beg) : 0;

        for (int jj = 0; jj < n_tiles; ++jj) {
            const int j = j_beg + jj;
            const bool cached = j < ep.n_ctiles;
            // From the page words two warp-uniform masks: pages with padding, pages whose slot differs from the
            // page before.  The pages of a new-token tile are masked from the causal limit of the tile's first row on.
            const int meta = meta_next;
            if (jj + 1 < n_tiles) meta_next = load_meta(j + 1);
            int prev = __shfl_up_sync(kFull, meta >> 8, 1);
            if (lane == 0) prev = cur_slot;
            const uint32_t chg_mask = __ballot_sync(kFull, (meta >> 8) != prev) & 0xffu;
            uint32_t mask_pages;
            int vis = kTileKeys;                                    // visible keys of this row in a new-token tile
            if (cached) {
                mask_pages = __ballot_sync(kFull, (meta & 0xff) < kPageTokens) & 0xffu;
            } else {
                const int kbase = (j - ep.n_ctiles) * kTileKeys;
                vis = c - kbase + 1;
                const int vis_lo = c_lo - kbase + 1;               // <= vis of every row of the tile
                mask_pages = vis_lo >= kTileKeys ? 0u : (0xffu << (max(vis_lo, 0) / kPageTokens)) & 0xffu;
            }

            ok = mbar_wait(bar_s_full(i), static_cast<uint32_t>(jj & 1), abort_flag, p.status);
            if (!ok) break;
            tc_fence_after();

            // the row's 128 scores
            uint32_t su[kTileKeys];
#pragma unroll
            for (int k = 0; k < 4; ++k)
                tmem_ld32_issue(t_s + static_cast<uint32_t>(k * 32), reinterpret_cast<uint32_t(&)[32]>(su[k * 32]));
            tmem_ld_wait();
#pragma unroll
            for (int k = 0; k < 4; ++k) tmem_ld32_arrived(reinterpret_cast<uint32_t(&)[32]>(su[k * 32]));
            float s[kTileKeys];
#pragma unroll
            for (int x = 0; x < kTileKeys; ++x) s[x] = __uint_as_float(su[x]);

            // hide page padding / keys after the causal limit
            for (uint32_t todo = mask_pages; todo; todo &= todo - 1u) {
                const int e = __ffs(static_cast<int>(todo)) - 1;    // warp-uniform
                const int nv_e = __shfl_sync(kFull, meta & 0xff, e);
                const int bound = cached ? nv_e : vis - e * kPageTokens;
                switch (e) {
#define ENL_MASK_PAGE(E)                                                          \
                    case E:                                                       \
                        _Pragma("unroll") for (int x = 0; x < kPageTokens; ++x)   \
                            if (x >= bound) s[E * kPageTokens + x] = kNegInf;     \
                        break;
                    ENL_MASK_PAGE(0) ENL_MASK_PAGE(1) ENL_MASK_PAGE(2) ENL_MASK_PAGE(3)
                    ENL_MASK_PAGE(4) ENL_MASK_PAGE(5) ENL_MASK_PAGE(6) ENL_MASK_PAGE(7)
#undef ENL_MASK_PAGE
                }
            }

            // row maximum: eight independent chains
            float mx8[kPagesPerTile];
#pragma unroll
            for (int k = 0; k < kPagesPerTile; ++k) {
                float a = fmax3(s[k * 16], s[k * 16 + 1], s[k * 16 + 2]);
#pragma unroll
                for (int x = 3; x < 15; x += 2) a = fmax3(a, s[k * 16 + x], s[k * 16 + x + 1]);
                mx8[k] = fmaxf(a, s[k * 16 + 15]);
            }
            const float m_cand = fmax3(fmax3(mx8[0], mx8[1], mx8[2]), fmax3(mx8[3], mx8[4], mx8[5]), fmaxf(mx8[6], mx8[7])) * scale;

            // The reference moves only when the row maximum has grown by more than the threshold (probabilities
            // stay below 2^threshold meanwhile); then the sums and the accumulator O_i are rescaled.  O_i holds
            // the tiles so far and no MMA touches it now: S_i of this tile completed after P_i V of the previous.
            const bool need = m_cand > m + kRescaleThreshold;       // also true when m == -inf < m_cand
            if (__any_sync(kFull, need)) {
                const float m_new = fmaxf(m, m_cand);
                const float alpha = (m_new == kNegInf) ? 1.f : ex2(m - m_new);
                l *= alpha;
                acc *= alpha;
                m = m_new;
                if (jj > 0) {
#pragma unroll 1
                    for (int k = 0; k < D / 32; ++k) {
                        uint32_t o[32];
                        tmem_ld32_wait(t_o + static_cast<uint32_t>(k * 32), o);
#pragma unroll
                        for (int x = 0; x < 32; ++x) o[x] = __float_as_uint(__uint_as_float(o[x]) * alpha);
                        tmem_st32(t_o + static_cast<uint32_t>(k * 32), o);
                    }
                }
            }
            const float m_use = (m == kNegInf) ? 0.f : m;

            // p = exp2(s * scale - m) in fp32; bf16 pairs (even key in the low half) into P_i, 32 keys per store, handed
            // to the MMA warp in two halves.  The page sums (of the fp32 values) are taken along the way: their adds
            // fill issue slots that the exponentials leave free.
            const uint64_t sc2 = pack2(scale, scale), nm2 = pack2(-m_use, -m_use);
            uint64_t ps2[kPagesPerTile];
#pragma unroll
            for (int ch = 0; ch < 4; ++ch) {
                uint32_t pk[16];
#pragma unroll
                for (int x = 0; x < 16; ++x) {
                    const int e = ch * 2 + (x >> 3);
                    float a0, a1;
                    unpack2(fma2(pack2(s[ch * 32 + 2 * x], s[ch * 32 + 2 * x + 1]), sc2, nm2), a0, a1);
                    a0 = ex2(a0);
                    a1 = ex2(a1);
                    const uint64_t p2 = pack2(a0, a1);
                    pk[x] = bf16x2(a0, a1);
                    ps2[e] = (x & 7) ? add2(ps2[e], p2) : p2;
                }
                tmem_st16(t_s + static_cast<uint32_t>(ch * 16), pk);
                if (ch & 1) {
                    tmem_st_wait();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_p_half(i, ch >> 1));
                }
            }

            // under the MMAs: row sum, slots
            float ps[kPagesPerTile];
#pragma unroll
            for (int e = 0; e < kPagesPerTile; ++e) {
                float lo, hi;
                unpack2(ps2[e], lo, hi);
                ps[e] = lo + hi;
            }
            const float tot = ((ps[0] + ps[1]) + (ps[2] + ps[3])) + ((ps[4] + ps[5]) + (ps[6] + ps[7]));
            l += tot;
            if (chg_mask == 0u) {
                acc += tot;
            } else {
#pragma unroll
                for (int e = 0; e < kPagesPerTile; ++e) {
                    if ((chg_mask >> e) & 1u) {
                        park(m_use);
                        acc = 0.f;
                        cur_slot = __shfl_sync(kFull, meta >> 8, e);
                    }
                    acc += ps[e];
                }
            }
        }

        // ---- per-row results ----
        const float m_use = (m == kNegInf) ? 0.f : m;
        const float lse = (l > 0.f) ? m_use + lg2(l) : kNegInf;
        // (row, head) index of row rr of this warp, or -1 beyond the episode's queries
        auto row_index = [&](int rr) -> int {
            const int r2 = q4 * 32 + rr;
            const int t2 = it.t0 + i * tile_tokens + r2 / rep;
            if (t2 >= ep.n_q) return -1;
            const int g2 = ep.q_off + t2;
            return (split_mode ? it.split * p.n_q_total + g2 : g2) * p.Hq + it.kvh * rep + r2 % rep;
        };
        // The warp's 32 rows x 128 bytes leave through the (idle) shared memory of the Q tile: row-per-thread
        // stores would touch 32 different rows per instruction.  Each thread stages its own 128 bytes, 16-byte
        // chunks swizzled by row, and the warp writes four whole row pieces per instruction.
        int ridx8[8];
#pragma unroll
        for (int itr = 0; itr < 8; ++itr) ridx8[itr] = row_index(itr * 4 + (lane >> 3));
        uint8_t *stg = smem + i * C::kTileBytes + q4 * 4096;
        auto flush_piece = [&](const uint32_t (&w)[32], uint8_t *gbase, long long row_pitch, int piece) {
#pragma unroll
            for (int cch = 0; cch < 8; ++cch)
                *reinterpret_cast<uint4 *>(stg + lane * 128 + ((cch ^ (lane & 7)) << 4)) =
                    make_uint4(w[4 * cch], w[4 * cch + 1], w[4 * cch + 2], w[4 * cch + 3]);
            __syncwarp();
#pragma unroll
            for (int itr = 0; itr < 8; ++itr) {
                const int rr = itr * 4 + (lane >> 3), cch = lane & 7;
                const uint4 v = *reinterpret_cast<const uint4 *>(stg + rr * 128 + ((cch ^ (rr & 7)) << 4));
                if (ridx8[itr] >= 0)
                    *reinterpret_cast<uint4 *>(gbase + ridx8[itr] * row_pitch + piece * 128 + cch * 16) = v;
            }
            __syncwarp();
        };
        // Masses: parked log-sums -> shares of the row's total.  ref / extra: per row (held by the row's thread) the
        // log-sum-exp of the whole row and, in a pair, the other split's part of the slot in which the splits meet.
        // Few slots: they were parked in shared memory.  Otherwise (the scoring pass has a thousand slots) the warp takes
        // 32 slots at a time, lanes over the slots (coalesced), the loads of all its 32 rows in flight together: the
        // cost is one memory round trip (some 3000 cycles while other CTAs stream their keys) per 32 slots; three
        // such chunks in flight at once measured slower.  Up to eight slots left over at the end (the new tokens'
        // slot after 64 groups, say) are taken row by lane instead, each thread converting its own row; their loads
        // are in flight with the first chunk's.
        // With mass_sum (Sec. 3.3 consumes only averages over an object's tokens and the q heads) the masses of the
        // warp's rows that belong to one object are added up on the way, lane by slot, and leave as one atomic add per
        // object and slot.
        const int my_ridx = row_index(lane);
        const int my_obj = (p.mass_sum && row_valid) ? __ldg(p.row_obj + grow) : -1;
        auto finish_masses = [&](float ref_mine, float extra_mine, int first, int last) {
            if (park_smem) {                                        // every thread converts its own row out of shared memory
                if (my_ridx < 0) return;
                float *slots = p.mass + static_cast<long long>(my_ridx) * p.mass_stride;
                float *sums = my_obj >= 0 ? p.mass_sum + static_cast<long long>(my_obj) * p.sum_stride : nullptr;
#pragma unroll 4
                for (int sl = first; sl <= last; ++sl) {
                    if (sl == skip_slot) continue;
                    float w = (ref_mine != kNegInf) ? ex2(park_row[sl * 128] - ref_mine) : 0.f;
                    if (sl == shared_slot && ref_mine != kNegInf) w += ex2(extra_mine - ref_mine);
                    slots[sl] = w;
                    if (sums) atomicAdd(sums + sl, w);
                }
                return;
            }
            __syncwarp();                                           // the parked values of all lanes are visible
            const int n_left = (last - first + 1) & 31;
            const int n_tail = (!p.mass_sum && n_left <= 8) ? n_left : 0;
            const int last_wide = last - n_tail;
            float *tail_slots = p.mass + static_cast<long long>(my_ridx) * p.mass_stride + last_wide + 1;
            float tv[8];
#pragma unroll
            for (int x = 0; x < 8; ++x)
                tv[x] = (x < n_tail && my_ridx >= 0 && last_wide + 1 + x != skip_slot) ? __ldcg(tail_slots + x) : kNegInf;
            constexpr int kChunks = 1;                              // 32-slot chunks whose loads are in flight together
#pragma unroll 1
            for (int sb = first + lane; sb - lane <= last_wide; sb += 32 * kChunks) {
              float v[kChunks][32];
#pragma unroll
              for (int ck = 0; ck < kChunks; ++ck) {
                const int s0 = sb + 32 * ck;
                const bool mine = s0 <= last_wide && s0 != skip_slot;
#pragma unroll
                for (int x = 0; x < 32; ++x) {
                    const int ri = __shfl_sync(kFull, my_ridx, x);
                    v[ck][x] = (mine && ri >= 0) ? __ldcg(p.mass + static_cast<long long>(ri) * p.mass_stride + s0) : kNegInf;
                }
              }
#pragma unroll
              for (int ck = 0; ck < kChunks; ++ck) {
                const int s0 = sb + 32 * ck;
                if (s0 - lane > last_wide) break;                   // warp-uniform
                const bool mine = s0 <= last_wide && s0 != skip_slot;
                float run = 0.f;                                    // this slot's sum over the rows of the current object
                int run_obj = -1;
#pragma unroll
                for (int x = 0; x < 32; ++x) {
                    const int ri = __shfl_sync(kFull, my_ridx, x);
                    const float ref = __shfl_sync(kFull, ref_mine, x);
                    const float extra = (shared_slot >= 0) ? __shfl_sync(kFull, extra_mine, x) : kNegInf;   // the same in all lanes
                    float w = 0.f;
                    if (mine && ri >= 0) {
                        w = (ref != kNegInf) ? ex2(v[ck][x] - ref) : 0.f;
                        if (s0 == shared_slot && ref != kNegInf) w += ex2(extra - ref);
                        p.mass[static_cast<long long>(ri) * p.mass_stride + s0] = w;
                    }
                    if (p.mass_sum) {                               // warp-uniform: obj is the same in every lane
                        const int obj = __shfl_sync(kFull, my_obj, x);
                        if (obj != run_obj) {
                            if (run_obj >= 0 && mine)
                                atomicAdd(p.mass_sum + static_cast<long long>(run_obj) * p.sum_stride + s0, run);
                            run = 0.f;
                            run_obj = obj;
                        }
                        run += w;
                    }
                }
                if (run_obj >= 0 && mine) atomicAdd(p.mass_sum + static_cast<long long>(run_obj) * p.sum_stride + s0, run);
              }
            }
            if (n_tail > 0 && my_ridx >= 0) {
#pragma unroll
                for (int x = 0; x < 8; ++x) {
                    const int sl = last_wide + 1 + x;
                    if (x >= n_tail || sl == skip_slot) continue;
                    float w = (ref_mine != kNegInf) ? ex2(tv[x] - ref_mine) : 0.f;
                    if (sl == shared_slot && ref_mine != kNegInf) w += ex2(extra_mine - ref_mine);
                    tail_slots[x] = w;
                }
            }
        };
        // slots this CTA walked (all of them without splits)
        int first_slot = 0, last_slot = G;
        if (p.n_splits > 1) {
            first_slot = G + 1;
            last_slot = -1;
            if (n_tiles > 0) {
                first_slot = (j_beg < ep.n_ctiles) ? (__ldg(p.stream_meta + ep.stream_off + j_beg * kPagesPerTile) >> 8) : G;
                last_slot = (j_end > ep.n_ctiles) ? G : (__ldg(p.stream_meta + ep.stream_off + j_end * kPagesPerTile - 1) >> 8);
            }
        }

        bool exported = false;
        if (ok) {
            park(m_use);
            if (!pair && !split_mode) {
                // ---- the whole key stream was this CTA's: output and masses ----
                if (p.mass) finish_masses(lse, kNegInf, 0, G);
                if (n_tiles > 0 && !p.mass_only) {
                    const float inv = (l > 0.f) ? 1.f / l : 0.f;
                    ok = mbar_wait(bar_o_done(i), 0, abort_flag, p.status);
                    if (ok) {
                        tc_fence_after();
#pragma unroll 1
                        for (int pc = 0; pc < D / 64; ++pc) {        // 64 bf16 channels = 128 bytes per row and piece
                            uint32_t o[32], w[32];
#pragma unroll
                            for (int k = 0; k < 2; ++k) {
                                tmem_ld32_wait(t_o + static_cast<uint32_t>(pc * 64 + k * 32), o);
#pragma unroll
                                for (int x = 0; x < 16; ++x)
                                    w[k * 16 + x] = bf16x2(__uint_as_float(o[2 * x]) * inv, __uint_as_float(o[2 * x + 1]) * inv);
                            }
                            flush_piece(w, static_cast<uint8_t *>(p.out), D * 2, pc);
                        }
                    }
                }
            } else if (split_mode) {
                // ---- partial results for the merge kernel: O / l in fp32, the row's log-sum-exp, raw slot log-sums ----
                if (row_valid) p.part_lse[rh] = lse;
                if (p.part_slot && park_smem) {
                    if (slot_out)
                        for (int sl = 0; sl <= G; ++sl)
                            slot_out[sl] = (sl < first_slot || sl > last_slot) ? kNegInf : park_row[sl * 128];
                } else if (p.part_slot) {
                    __syncwarp();
#pragma unroll 1
                    for (int rr = 0; rr < 32; ++rr) {               // slots this split did not walk contribute nothing
                        const int ri = __shfl_sync(kFull, my_ridx, rr);
                        if (ri < 0) continue;
                        float *slots = p.part_slot + static_cast<long long>(ri) * p.mass_stride;
                        for (int sl = lane; sl <= G; sl += 32)
                            if (sl < first_slot || sl > last_slot) slots[sl] = kNegInf;
                    }
                }
                if (n_tiles > 0) {
                    const float inv = (l > 0.f) ? 1.f / l : 0.f;
                    ok = mbar_wait(bar_o_done(i), 0, abort_flag, p.status);
                    if (ok) {
                        tc_fence_after();
#pragma unroll 1
                        for (int pc = 0; pc < D / 32; ++pc) {        // 32 fp32 channels = 128 bytes per row and piece
                            uint32_t o[32];
                            tmem_ld32_wait(t_o + static_cast<uint32_t>(pc * 32), o);
#pragma unroll
                            for (int x = 0; x < 32; ++x) o[x] = __float_as_uint(__uint_as_float(o[x]) * inv);
                            flush_piece(o, reinterpret_cast<uint8_t *>(p.part_o), D * 4, pc);
                        }
                    }
                }
            } else {
              if constexpr (D == 128) {
                // ---- pair merge: the two CTAs of the cluster hold the two halves of the key stream ----
                const uint32_t peer = cluster_rank() ^ 1u;
                // they tell each other (reference, sum, shared-slot part) of every row
                {
                    const uint32_t mine = sbase + static_cast<uint32_t>(C::kXpeerOff + (i * 128 + r) * 16);
                    peer_push4(peer_addr(mine, peer), m_use, l, bnd, 0.f, peer_addr(bar_peer_ml, peer));
                }
                constexpr uint32_t kRingOff = kQTiles * C::kTileBytes;
                constexpr uint32_t kExportStageOff = 65536;         // upper half of the ring (4 stages x 32 KB)
                const uint32_t warp_off = kRingOff + static_cast<uint32_t>(q4 * 16384);
                if (i != it.split && n_tiles > 0) {
                    // This CTA finishes Q tile `it.split`; the accumulator of the other tile goes to the peer, which
                    // finishes that one.  It goes as it is (relative to this CTA's own reference; the peer learns the
                    // weight from the row sums above), so that nothing but the last MMA stands before it: staged
                    // row-per-thread in the upper half of this CTA's ring (idle once both tiles' MMAs are done; 16 KB
                    // per warp, 16-byte chunks swizzled by row), then one bulk copy per warp into the lower half of
                    // the peer's ring, counted in bytes on the peer's barrier.
                    ok = mbar_wait(bar_o_done(i), 0, abort_flag, p.status);
                    if (ok && n_qt == 2) ok = mbar_wait(bar_o_done(i ^ 1), 0, abort_flag, p.status);
                    if (ok) {
                        tc_fence_after();
                        uint8_t *stage = smem + warp_off + kExportStageOff + lane * 512;
#pragma unroll 1
                        for (int k = 0; k < 4; ++k) {
                            uint32_t o[32];
                            tmem_ld32_wait(t_o + static_cast<uint32_t>(k * 32), o);
#pragma unroll
                            for (int cch = 0; cch < 8; ++cch)
                                *reinterpret_cast<uint4 *>(stage + (((k * 8 + cch) ^ (lane & 7)) << 4)) =
                                    make_uint4(o[4 * cch], o[4 * cch + 1], o[4 * cch + 2], o[4 * cch + 3]);
                        }
                        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                        __syncwarp();
                        ok = mbar_wait<true>(bar_peer_free, 0, abort_flag, p.status);
                        if (ok && lane == 0)
                            peer_bulk_copy(peer_addr(sbase + warp_off, peer), sbase + warp_off + kExportStageOff, 16384,
                                           peer_addr(bar_peer_o, peer));
                        exported = ok;
                    }
                }
                // the merged row: reference, sum, weights of the two accumulators
                float pair_lse = kNegInf, pair_bnd = kNegInf, w_own = 0.f, w_peer = 0.f;
                if (ok) ok = mbar_wait<true>(bar_peer_ml, 0, abort_flag, p.status);
                if (ok) {
                    const float4 pe = *reinterpret_cast<const float4 *>(smem + C::kXpeerOff + (i * 128 + r) * 16);
                    const bool va = l > 0.f, vb = pe.y > 0.f;
                    const float M = fmaxf(va ? m_use : kNegInf, vb ? pe.x : kNegInf);
                    const float fa = va ? ex2(m_use - M) : 0.f;
                    const float fb = vb ? ex2(pe.x - M) : 0.f;
                    const float L = (va ? l * fa : 0.f) + (vb ? pe.y * fb : 0.f);
                    pair_lse = (L > 0.f) ? M + lg2(L) : kNegInf;
                    pair_bnd = pe.z;
                    w_own = (L > 0.f) ? fa / L : 0.f;
                    w_peer = (L > 0.f) ? fb / L : 0.f;
                }
                // each CTA writes the slots it walked against the merged log-sum-exp; the slot both walked is
                // written by split 0, which adds the part split 1 sent.  (Before the output: the peer's accumulator is
                // still on its way.)
                if (ok && p.mass) finish_masses(pair_lse, pair_bnd, first_slot, last_slot);
                if (ok && i == it.split && n_tiles > 0) {
                    // this CTA finishes the tile: its own accumulator and what the peer sent, each with its weight;
                    // thread (warp, lane) reads what thread (warp, lane) of the peer wrote
                    ok = mbar_wait(bar_o_done(i), 0, abort_flag, p.status);
                    if (ok) {
                        tc_fence_after();
                        ok = mbar_wait<true>(bar_peer_o, 0, abort_flag, p.status);
                        // the peer may retire once its staging area has been read out: tell it
                        if (ok && q4 == 0 && lane == 0) peer_arrive_relaxed(peer_addr(bar_peer_ack, peer));
                    }
                    if (ok) {
                        const uint8_t *theirs = smem + warp_off + lane * 512;
#pragma unroll 1
                        for (int pc = 0; pc < 2; ++pc) {
                            uint32_t o[32], w[32];
#pragma unroll
                            for (int k = 0; k < 2; ++k) {
                                tmem_ld32_wait(t_o + static_cast<uint32_t>(pc * 64 + k * 32), o);
#pragma unroll
                                for (int cch = 0; cch < 8; ++cch) {
                                    const float4 a = *reinterpret_cast<const float4 *>(
                                        theirs + ((((pc * 2 + k) * 8 + cch) ^ (lane & 7)) << 4));
                                    auto mix = [&](uint32_t own, float th) { return fmaf(__uint_as_float(own), w_own, th * w_peer); };
                                    w[k * 16 + 2 * cch] = bf16x2(mix(o[4 * cch], a.x), mix(o[4 * cch + 1], a.y));
                                    w[k * 16 + 2 * cch + 1] = bf16x2(mix(o[4 * cch + 2], a.z), mix(o[4 * cch + 3], a.w));
                                }
                            }
                            flush_piece(w, static_cast<uint8_t *>(p.out), D * 2, pc);
                        }
                    }
                }
                // what this CTA staged for its peer must have been fetched before the CTA may retire
                if (exported) ok = mbar_wait<true>(bar_peer_ack, 0, abort_flag, p.status);
              }
            }
        }
      }
    }

    // ---- teardown ----
    tc_fence_before();
    __syncthreads();
    if (warp == kMmaWarp) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

}  // namespace

size_t attention_smem_bytes(int head_dim)
{
    return head_dim == 128 ? Cfg<128>::kSmemBytes : Cfg<64>::kSmemBytes;
}

cudaError_t prepare_attention(int head_dim)
{
    if (head_dim == 128)
        return cudaFuncSetAttribute(attn_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<128>::kSmemBytes);
    if (head_dim == 64)
        return cudaFuncSetAttribute(attn_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<64>::kSmemBytes);
    return cudaErrorInvalidValue;
}

bool attention_pairs_supported()
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = Cfg<128>::kSmemBytes;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, attn_kernel<128>, &cfg) != cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    return n > 0;
}

cudaError_t launch_attention(const AttnParams &p, int head_dim, int n_items, cudaStream_t st)
{
    if (n_items <= 0) return cudaSuccess;
    cudaError_t e;
    if (p.pair_merge && (head_dim != 128 || p.n_splits != 2 || (n_items & 1))) return cudaErrorInvalidValue;
    if (head_dim == 128)
        e = launch_pdl(attn_kernel<128>, dim3(n_items), dim3(kThreads), Cfg<128>::kSmemBytes, st, p, p.pair_merge ? 2u : 1u);
    else if (head_dim == 64)
        e = launch_pdl(attn_kernel<64>, dim3(n_items), dim3(kThreads), Cfg<64>::kSmemBytes, st, p);
    else
        return cudaErrorInvalidValue;
    return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace enl
