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
// to; when a slot ends its log2-sum-exp is parked in the mass buffer, and after the last tile the row
// turns those into probabilities.  With KV splits every split writes partial results that a second
// kernel merges.
//
// Roles: 16 softmax warps -- Q tile i = warps 8i..8i+7, and within a tile warps 0-3 take key columns 0..63
// of every S tile ("half A"), warps 4-7 columns 64..127 ("half B"), so that every row is shared by two
// threads of two warps with the same TMEM lane quadrant; they exchange the row maximum (and half B's page
// sums, which half A credits to the slots) through shared memory behind a two-warp mbarrier.  Four
// softmax warps per scheduler overlap each other's exp2, max, pack and TMEM traffic.  Warp 16 is the TMA
// producer, warp 17 the MMA issuer (and TMEM owner), warps 18-19 idle: they complete the fifth warpgroup
// so that setmaxnreg can move registers to the softmax warpgroups.
// TMEM columns: S0 [0,128) S1 [128,256) O0 [256,384) O1 [384,512); P_i (bf16) overwrites columns [0,32) and
// [64,96) of S_i, each softmax half inside its own columns.
#include <cuda_bf16.h>

#include "enl_internal.h"
#include "tmem_ops.cuh"

namespace enl {
namespace {

constexpr int kThreads      = 640;
constexpr int kSoftmaxWarps = 16;
constexpr int kRegsSoftmax  = 104;            // the launch gives 640 x 96 registers; what warpgroup 4 releases (4 x 8 per thread) is what the four softmax warpgroups gain
constexpr int kRegsOther    = 64;
constexpr int kProducerWarp = 16;
constexpr int kMmaWarp      = 17;
constexpr uint32_t kTmemCols = 512;
constexpr float kRescaleThreshold = 8.0f;     // log2 units: p stays below 2^8 between max updates
constexpr float kMaxJump = 100.0f;            // log2 units: most a tile's scores may exceed the maximum of all earlier tiles
constexpr unsigned long long kWaitLimitNs = 1000ull * 1000ull * 1000ull;

template <int D>
struct Cfg {
    static constexpr int kHalves    = D / 64;             // 64-channel (128-byte) column blocks
    static constexpr int kHalfBytes = 128 * 128;          // 128 rows x 128 B
    static constexpr int kTileBytes = kHalves * kHalfBytes;
    static constexpr int kStages    = (D == 128) ? 4 : 8;
    static constexpr int kBarOff    = (kQTiles + kStages) * kTileBytes;
    // exchange area of the softmax thread pairs: row maxima [parity][tile][half][128], page sums
    // [tile mod 3][tile][8 pages][128], 1 / row sum [tile][128]
    static constexpr int kXmaxOff   = kBarOff + 512;
    static constexpr int kXsumOff   = kXmaxOff + 2 * kQTiles * 2 * 128 * 4;
    static constexpr int kXinvOff   = kXsumOff + 3 * kQTiles * kPagesPerTile * 128 * 4;
    // pair merge: what the other CTA of the cluster knows about this CTA's rows, [tile][128] x (m, l, shared-slot log-sum, -)
    static constexpr int kXpeerOff  = kXinvOff + kQTiles * 128 * 4;
    static constexpr int kSmemBytes = kXpeerOff + kQTiles * 128 * 16 + 1024;   // + alignment slack
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
    bool ok = poll();
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
    return __all_sync(0xffffffffu, ok);
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
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after()  { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]
__device__ __forceinline__ void mma_ss(uint32_t d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]
__device__ __forceinline__ void mma_ts(uint32_t d, uint32_t a, uint64_t bdesc, uint32_t idesc, uint32_t acc)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d), "r"(a), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
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

// Optional phase timestamps of CTA 0 (development builds only; never compiled into the library).
#ifdef ENL_TRACE
__device__ long long g_trace[5][96][8];
#define ENL_TR(role, tile, slot) do { if (blockIdx.x == 0 && lane == 0 && (tile) < 96) g_trace[role][tile][slot] = clock64(); } while (0)
#define ENL_PIN(x) asm volatile("" : "+f"(x) :: "memory")
#else
#define ENL_TR(role, tile, slot) do { } while (0)
#define ENL_PIN(x) do { } while (0)
#endif

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
    auto bar_p_full   = [&](int i) { return bar0 + 8u * (3 + 2 * C::kStages + i); };
    auto bar_o_done   = [&](int i) { return bar0 + 8u * (5 + 2 * C::kStages + i); };
    auto bar_pair     = [&](int k) { return bar0 + 8u * (7 + 2 * C::kStages + k); };   // k = tile * 4 + lane quadrant
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + C::kBarOff + 8 * (15 + 2 * C::kStages));
    // pair merge (cluster of two): the peer's row sums have arrived / the peer's partial output has arrived /
    // the peer's K/V ring is idle and may be written
    const uint32_t bar_peer_ml = bar0 + 8u * (16 + 2 * C::kStages);
    const uint32_t bar_peer_o = bar0 + 8u * (17 + 2 * C::kStages);
    const uint32_t bar_peer_free = bar0 + 8u * (18 + 2 * C::kStages);
    const uint32_t bar_peer_ack = bar0 + 8u * (19 + 2 * C::kStages);   // the peer has received what this CTA staged for it
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
            mbar_init(bar_p_full(i), 8);          // one arrival per softmax warp of the tile
            mbar_init(bar_o_done(i), 1);
        }
        for (int k = 0; k < 4 * kQTiles; ++k) mbar_init(bar_pair(k), 2);
        mbar_init(bar_peer_ml, 1);                                   // this thread's arrival below + 16 bytes per row from the peer
        mbar_init(bar_peer_o, 1);                                    // this thread's arrival below + 64 KB from the peer
        mbar_init(bar_peer_free, 1);
        mbar_init(bar_peer_ack, 1);
        if (p.pair_merge) {
            mbar_expect_tx(bar_peer_ml, static_cast<uint32_t>(n_qt * 128 * 16));
            mbar_expect_tx(bar_peer_o, 8u * 8192u);
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
            auto issue_qk = [&](int i, int st) {
                if (lane == 0) {
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk) {
                        const uint32_t off = static_cast<uint32_t>((kk >> 2) * C::kHalfBytes + (kk & 3) * 32);
                        mma_ss(tmem_s(i), smem_desc(q_addr(i) + off, 16), smem_desc(stage_addr(st) + off, 16),
                               idesc_qk, kk > 0 ? 1u : 0u);
                    }
                    tc_commit(bar_s_full(i));
                }
                __syncwarp();
            };
            auto issue_pv = [&](int i, int st, bool first_tile) {
                if (lane == 0) {
#pragma unroll
                    for (int kk = 0; kk < kTileKeys / 16; ++kk) {
                        mma_ts(tmem_o(i), tmem_s(i) + static_cast<uint32_t>((kk >> 2) * 64 + (kk & 3) * 8),   // P of keys 64.. sits in columns 64..
                               smem_desc(stage_addr(st) + static_cast<uint32_t>(kk * 16 * 128), C::kHalfBytes),
                               idesc_pv, (first_tile && kk == 0) ? 0u : 1u);
                    }
                }
                __syncwarp();
            };
            auto commit_to = [&](uint32_t bar) {
                if (lane == 0) tc_commit(bar);
                __syncwarp();
            };
            auto wait_full = [&](int f) {
                return mbar_wait(bar_kv_full(f % C::kStages), static_cast<uint32_t>((f / C::kStages) & 1),
                                 abort_flag, p.status);
            };

            ok = mbar_wait(bar_q_full, 0, abort_flag, p.status);
            if (ok) ok = wait_full(0);
            if (ok) {
                tc_fence_after();
                for (int i = 0; i < n_qt; ++i) issue_qk(i, 0);
                commit_to(bar_kv_empty(0));
            }
            for (int jj = 0; jj < n_tiles && ok; ++jj) {
                const int fv = 2 * jj + 1, fk = 2 * jj + 2;             // ring slots of V_jj and K_{jj+1}
                const bool more = jj + 1 < n_tiles;
                ok = wait_full(fv);
                if (ok && more) ok = wait_full(fk);
                if (!ok) break;
                for (int i = 0; i < n_qt; ++i) {
                    ENL_TR(4, jj, 4 * i);
                    ok = mbar_wait(bar_p_full(i), static_cast<uint32_t>(jj & 1), abort_flag, p.status);
                    if (!ok) break;
                    tc_fence_after();
                    ENL_TR(4, jj, 4 * i + 1);
                    issue_pv(i, fv % C::kStages, jj == 0);
                    if (i == n_qt - 1) commit_to(bar_kv_empty(fv % C::kStages));
                    if (!more) commit_to(bar_o_done(i));
                    if (more) {
                        issue_qk(i, fk % C::kStages);
                        if (i == n_qt - 1) commit_to(bar_kv_empty(fk % C::kStages));
                    }
                    ENL_TR(4, jj, 4 * i + 2);
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
      if ((warp >> 3) < n_qt) {
        // ================= softmax / epilogue: two threads per row, 64 key columns each =================
        constexpr int kHalfCols = kTileKeys / 2;                   // 64 key columns = 4 pages per thread
        constexpr int kHalfPages = kPagesPerTile / 2;
        const int i = warp >> 3;                                   // Q tile
        const int hb = (warp >> 2) & 1;                            // 0: columns 0..63 (owner of the row's sums), 1: 64..127
        const int q4 = warp & 3;                                   // TMEM lane quadrant
        const bool owner = hb == 0;
        const int r = q4 * 32 + lane;
        const int t = it.t0 + i * tile_tokens + r / rep;           // episode-relative query token
        const int h = it.kvh * rep + r % rep;
        const bool row_valid = t < ep.n_q;
        const int c = min(ep.n_new - ep.n_q + t, ep.n_new - 1);    // last visible new key
        const int G = ep.n_slots;
        const uint32_t lane_sel = static_cast<uint32_t>(q4 * 32) << 16;
        const uint32_t t_s = tmem_base + lane_sel + static_cast<uint32_t>(i * 128);
        const uint32_t t_o = tmem_base + lane_sel + static_cast<uint32_t>(256 + i * 128);
        const bool split_mode = p.n_splits > 1 && !pair;
        const long long grow = static_cast<long long>(ep.q_off) + t;   // global query row
        const long long rh = (split_mode ? (static_cast<long long>(it.split) * p.n_q_total + grow) : grow) * p.Hq + h;
        float *slot_out = nullptr;
        if (row_valid && owner) {
            if (split_mode) { if (p.part_slot) slot_out = p.part_slot + rh * p.mass_stride; }
            else if (p.mass) slot_out = p.mass + rh * p.mass_stride;
        }
        const float scale = p.scale_log2;
        const float inv_scale = 1.f / scale;
        float *xmax_own = reinterpret_cast<float *>(smem + C::kXmaxOff) + (i * 2 + hb) * 128 + r;          // + parity * kQTiles*2*128
        float *xmax_other = reinterpret_cast<float *>(smem + C::kXmaxOff) + (i * 2 + (hb ^ 1)) * 128 + r;
        constexpr int kXmaxPar = kQTiles * 2 * 128;
        float *xsum = reinterpret_cast<float *>(smem + C::kXsumOff) + i * (kPagesPerTile * 128) + r;   // + (tile mod 3) * kQTiles*8*128 + page*128
        float *xinv = reinterpret_cast<float *>(smem + C::kXinvOff) + i * 128 + r;
        const uint32_t pbar = bar_pair(i * 4 + q4);
        uint32_t n_sync = 0;
        // the two warps that share 32 rows meet here; bounded like every other wait
        auto pair_sync = [&]() -> bool {
            __syncwarp();
            if (lane == 0) mbar_arrive(pbar);
            const bool done = mbar_wait(pbar, n_sync & 1u, abort_flag, p.status);
            ++n_sync;
            return done;
        };

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
        float m = kNegInf, l = 0.f, acc = 0.f;                     // l, acc: owner only
        float mx_prev = kNegInf;                                   // this thread's maximum of the previous tile (unscaled)
        int cur_slot = -1;
        // a page's sum goes to its slot; a slot that ends parks its log2-sum-exp
        auto credit = [&](int slot, float v, float m_ref) {
            if (slot != cur_slot) {
                if (cur_slot == skip_slot) bnd = lg2(acc) + m_ref;
                else if (slot_out && cur_slot >= 0) slot_out[cur_slot] = lg2(acc) + m_ref;
                acc = 0.f;
                cur_slot = slot;
            }
            acc += v;
            l += v;
        };
        // The owner credits the eight page sums of tile j (its own four and half B's four, both parked in shared
        // memory) only after it has handed P of tile j + 1 to the MMA warp: the slot book-keeping and its
        // scattered stores then overlap the MMAs instead of delaying them.  `late` = the factor by which the
        // running sums were rescaled since those page sums were taken.
        auto credit_tile = [&](int jt, float late, float m_ref) {
            const float *src = xsum + (jt % 3) * (kQTiles * kPagesPerTile * 128);
            const int jg = j_beg + jt;
            if (jg < ep.n_ctiles) {
                const int4 *e4 = reinterpret_cast<const int4 *>(p.stream_meta + ep.stream_off + jg * kPagesPerTile);
                const int4 a = __ldg(e4), b = __ldg(e4 + 1);
                credit(a.x >> 8, src[0 * 128] * late, m_ref);
                credit(a.y >> 8, src[1 * 128] * late, m_ref);
                credit(a.z >> 8, src[2 * 128] * late, m_ref);
                credit(a.w >> 8, src[3 * 128] * late, m_ref);
                credit(b.x >> 8, src[4 * 128] * late, m_ref);
                credit(b.y >> 8, src[5 * 128] * late, m_ref);
                credit(b.z >> 8, src[6 * 128] * late, m_ref);
                credit(b.w >> 8, src[7 * 128] * late, m_ref);
            } else {
                float v = 0.f;
#pragma unroll
                for (int e = 0; e < kPagesPerTile; ++e) v += src[e * 128];
                credit(G, v * late, m_ref);
            }
        };

        for (int jj = 0; jj < n_tiles; ++jj) {
            const int j = j_beg + jj;
            // valid keys of this thread's four pages, one byte each: page padding (cached tiles) or the causal
            // limit (new-token tiles)
            uint32_t nvp;
            if (j < ep.n_ctiles) {
                const int4 mv = __ldg(reinterpret_cast<const int4 *>(p.stream_meta + ep.stream_off + j * kPagesPerTile) + hb);
                nvp = static_cast<uint32_t>(mv.x & 0xff) | (static_cast<uint32_t>(mv.y & 0xff) << 8) |
                      (static_cast<uint32_t>(mv.z & 0xff) << 16) | (static_cast<uint32_t>(mv.w & 0xff) << 24);
            } else {
                const int vis = c - (j - ep.n_ctiles) * kTileKeys - hb * kHalfCols + 1;   // visible keys of this half
                nvp = 0;
#pragma unroll
                for (int e = 0; e < kHalfPages; ++e)
                    nvp |= static_cast<uint32_t>(min(max(vis - e * kPageTokens, 0), kPageTokens)) << (8 * e);
            }
            if (q4 == 0) ENL_TR(warp >> 2, jj, 0);
            ok = mbar_wait(bar_s_full(i), static_cast<uint32_t>(jj & 1), abort_flag, p.status);
            if (!ok) break;
            tc_fence_after();
            if (q4 == 0) ENL_TR(warp >> 2, jj, 1);

            // hide page padding / keys after the causal limit of page e (16 scores), and take the page's maximum
            auto page_max = [&](int e, float (&sc)[kPageTokens]) -> float {
                const int nv = static_cast<int>((nvp >> (8 * e)) & 0xffu);
                if (nv < kPageTokens) {
#pragma unroll
                    for (int x = 0; x < kPageTokens; ++x)
                        if (x >= nv) sc[x] = kNegInf;
                }
                float a = fmax3(sc[0], sc[1], sc[2]);
#pragma unroll
                for (int x = 3; x < 15; x += 2) a = fmax3(a, sc[x], sc[x + 1]);
                return fmaxf(a, sc[15]);
            };
            const uint32_t t_half = t_s + static_cast<uint32_t>(hb * kHalfCols);

            // The reference maximum needs the other half's columns too.  Waiting for them every tile would put a
            // two-warp barrier on the critical path, so the exchange lags by one tile: this tile's exponentials
            // use the maximum over all EARLIER tiles (both halves know it: the partner's maximum of the previous
            // tile has been in shared memory since before that tile's P was handed over), and this tile's
            // maximum only moves the reference for the next one.  A probability may then exceed 1 by the factor
            // 2^(jump of this tile over everything before it), harmless in floating point up to kMaxJump.  The
            // first tile, and any tile that starts without a reference, need their own maximum first: a pass over
            // the scores for the maximum alone, exchanged synchronously.
            const bool sync_tile = (jj == 0) || __any_sync(0xffffffffu, m == kNegInf);   // same rows, same m in both halves
            float mx_ref;
            if (sync_tile) {
                float mx0 = kNegInf;
#pragma unroll 1
                for (int e = 0; e < kHalfPages; ++e) {
                    uint32_t su[kPageTokens];
                    tmem_ld16_wait(t_half + static_cast<uint32_t>(e * kPageTokens), su);
                    float sc[kPageTokens];
#pragma unroll
                    for (int x = 0; x < kPageTokens; ++x) sc[x] = __uint_as_float(su[x]);
                    mx0 = fmaxf(mx0, page_max(e, sc));
                }
                xmax_own[(jj & 1) * kXmaxPar] = mx0;
                ok = pair_sync();
                if (!ok) break;
                mx_ref = fmaxf(mx0, xmax_other[(jj & 1) * kXmaxPar]);
            } else {
                mx_ref = fmaxf(mx_prev, xmax_other[((jj - 1) & 1) * kXmaxPar]);
            }
            if (q4 == 0) ENL_TR(warp >> 2, jj, 2);

            float late = 1.f;
            const float m_cand = mx_ref * scale;
            const bool need = m_cand > m + kRescaleThreshold;       // also true when m == -inf < m_cand
            if (__any_sync(0xffffffffu, need)) {                     // same rows, same decision in both halves
                // the reference moves by at most kMaxJump per tile, so that the rescale factor cannot underflow
                // (only a row that has already been reported as out of range is ever held back by this)
                const float m_new = (m == kNegInf) ? m_cand : fminf(fmaxf(m, m_cand), m + kMaxJump);
                const float alpha = (m_new == kNegInf) ? 1.f : ex2(m - m_new);
                l *= alpha;
                acc *= alpha;
                late = alpha;
                m = m_new;
                if (jj > 0) {                                        // O_i holds the tiles so far; each half rescales D/2 columns
#pragma unroll 1
                    for (int k = 0; k < D / 32; ++k) {
                        uint32_t o[16];
                        const uint32_t col = static_cast<uint32_t>(hb * (D / 2) + k * 16);
                        tmem_ld16_wait(t_o + col, o);
#pragma unroll
                        for (int x = 0; x < 16; ++x) o[x] = __float_as_uint(__uint_as_float(o[x]) * alpha);
                        tmem_st16(t_o + col, o);
                    }
                }
            }
            const float m_use = (m == kNegInf) ? 0.f : m;
            const float cap = (m_use + kMaxJump) * inv_scale;       // largest score the reference can carry

            // The scores are taken page by page (16 per thread and load; the next page's load is in flight while
            // this one is worked on): mask, maximum (for the next tile's reference), p = exp2(s * scale - m).  The
            // page's sum goes to shared memory (the owner credits it to its slot later), its sixteen probabilities
            // go as eight bf16 pairs (even key in the low half) into P.  Each half keeps its P inside its own 64
            // columns of S_i: page e at columns hb*64 + 8e .. +7, which only covers scores already taken.
            const uint64_t sc2 = pack2(scale, scale), nm2 = pack2(-m_use, -m_use);
            float *sum_dst = xsum + (jj % 3) * (kQTiles * kPagesPerTile * 128) + hb * (kHalfPages * 128);
            float mx = kNegInf;
            uint32_t su[2][kPageTokens];
            tmem_ld16_issue(t_half, su[0]);
#pragma unroll
            for (int e = 0; e < kHalfPages; ++e) {
                tmem_ld16_arrived(su[e & 1]);
                if (e + 1 < kHalfPages) tmem_ld16_issue(t_half + static_cast<uint32_t>((e + 1) * kPageTokens), su[(e + 1) & 1]);
                float sc[kPageTokens];
#pragma unroll
                for (int x = 0; x < kPageTokens; ++x) sc[x] = __uint_as_float(su[e & 1][x]);
                const float pm = page_max(e, sc);
                mx = fmaxf(mx, pm);
                if (pm > cap) {
                    // beyond what the lagging reference can carry: keep the result finite and report it
                    atomicExch(p.status, 3);
#pragma unroll
                    for (int x = 0; x < kPageTokens; ++x) sc[x] = fminf(sc[x], cap);
                }
                uint64_t pr[kPageTokens / 2];
                uint32_t pk[kPageTokens / 2];
#pragma unroll
                for (int x = 0; x < kPageTokens / 2; ++x) {
                    float a0, a1;
                    unpack2(fma2(pack2(sc[2 * x], sc[2 * x + 1]), sc2, nm2), a0, a1);
                    a0 = ex2(a0);
                    a1 = ex2(a1);
                    pr[x] = pack2(a0, a1);
                    const __nv_bfloat162 bb = __floats2bfloat162_rn(a0, a1);
                    pk[x] = *reinterpret_cast<const uint32_t *>(&bb);
                }
                tmem_st8(t_s + static_cast<uint32_t>(hb * kHalfCols + e * 8), pk);
                const uint64_t q0 = add2(add2(pr[0], pr[1]), add2(pr[2], pr[3]));
                const uint64_t q1 = add2(add2(pr[4], pr[5]), add2(pr[6], pr[7]));
                float b0, b1;
                unpack2(add2(q0, q1), b0, b1);
                sum_dst[e * 128] = b0 + b1;
            }
            if (!sync_tile) xmax_own[(jj & 1) * kXmaxPar] = mx;     // (a synchronous tile has published it already)
            mx_prev = mx;
            if (q4 == 0) ENL_TR(warp >> 2, jj, 3);
            tmem_st_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_p_full(i));
            if (q4 == 0) ENL_TR(warp >> 2, jj, 4);
            if (owner && jj > 0) credit_tile(jj - 1, late, m_use);
        }

        // ---- per-row results ----
        float m_use = (m == kNegInf) ? 0.f : m;
        bool exported = false;
        float w_peer = 0.f;
        if (ok) ok = pair_sync();                                   // half B's sums of the last tile are in place
        if (ok) {
            if (owner && n_tiles > 0) credit_tile(n_tiles - 1, 1.f, m_use);
            const float inv = (l > 0.f) ? 1.f / l : 0.f;
            float pair_lse = kNegInf, pair_bnd = kNegInf;
            const float lse = (l > 0.f) ? m_use + lg2(l) : kNegInf;
            if (owner) {
                if (cur_slot == skip_slot && cur_slot >= 0) bnd = lg2(acc) + m_use;
                else if (slot_out && cur_slot >= 0) slot_out[cur_slot] = lg2(acc) + m_use;
                if (pair) {
                    // the two CTAs of the cluster tell each other (reference, sum, shared-slot part) of every row
                    const uint32_t peer = cluster_rank() ^ 1u;
                    const uint32_t mine = sbase + static_cast<uint32_t>(C::kXpeerOff + (i * 128 + r) * 16);
                    peer_push4(peer_addr(mine, peer), m_use, l, bnd, 0.f, peer_addr(bar_peer_ml, peer));
                }
            }
            if constexpr (D == 128) {
              if (pair && i != it.split && n_tiles > 0) {
                // This CTA finishes Q tile `it.split`; the accumulator of the other tile goes to the peer, which
                // finishes that one.  It goes as it is (relative to this CTA's own reference; the peer learns the
                // weight from the row sums above), so that nothing but the last MMA stands before it: staged
                // row-per-thread in the upper half of this CTA's ring (idle once both tiles' MMAs are done; 8 KB per
                // warp, 16-byte chunks swizzled by row), then one bulk copy per warp into the lower half of the
                // peer's ring, counted in bytes on the peer's barrier.
                const uint32_t peer = cluster_rank() ^ 1u;
                const uint32_t warp_off = static_cast<uint32_t>(kQTiles * C::kTileBytes + (hb * 4 + q4) * 8192);
                constexpr uint32_t kExportStageOff = 65536;         // upper half of the ring (4 stages x 32 KB)
                ok = mbar_wait(bar_o_done(i), 0, abort_flag, p.status);
                if (ok && n_qt == 2) ok = mbar_wait(bar_o_done(i ^ 1), 0, abort_flag, p.status);
                if (ok) {
                    tc_fence_after();
                    uint8_t *stage = smem + warp_off + kExportStageOff + lane * 256;
#pragma unroll 1
                    for (int k = 0; k < 2; ++k) {
                        uint32_t o[32];
                        tmem_ld32_wait(t_o + static_cast<uint32_t>(hb * (D / 2) + k * 32), o);
#pragma unroll
                        for (int cch = 0; cch < 8; ++cch)
                            *reinterpret_cast<uint4 *>(stage + (((k * 8 + cch) ^ (lane & 7)) << 4)) =
                                make_uint4(o[4 * cch], o[4 * cch + 1], o[4 * cch + 2], o[4 * cch + 3]);
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    ok = mbar_wait<true>(bar_peer_free, 0, abort_flag, p.status);
                    if (ok && lane == 0)
                        peer_bulk_copy(peer_addr(sbase + warp_off, peer), sbase + warp_off + kExportStageOff, 8192,
                                       peer_addr(bar_peer_o, peer));
                    exported = ok;
                }
              }
            }
            if (owner && ok) {
                if (pair) {
                    ok = mbar_wait<true>(bar_peer_ml, 0, abort_flag, p.status);
                    const float4 pe = *reinterpret_cast<const float4 *>(smem + C::kXpeerOff + (i * 128 + r) * 16);
                    const bool va = l > 0.f, vb = pe.y > 0.f;
                    const float M = fmaxf(va ? m_use : kNegInf, vb ? pe.x : kNegInf);
                    const float fa = va ? ex2(m_use - M) : 0.f;
                    const float L = (va ? l * fa : 0.f) + (vb ? pe.y * ex2(pe.x - M) : 0.f);
                    pair_lse = (L > 0.f) ? M + lg2(L) : kNegInf;
                    pair_bnd = pe.z;
                    *xinv = (L > 0.f) ? fa / L : 0.f;                // weight of this CTA's unnormalised O
                    w_peer = (L > 0.f && vb) ? ex2(pe.x - M) / L : 0.f;   // and of the peer's
                    xmax_other[0] = w_peer;                          // for half B (its slot of the exchange area is idle)
                } else if (split_mode) {
                    if (row_valid) {
                        // slots this split did not walk contribute nothing
                        int first = G + 1, last = -1;
                        if (n_tiles > 0) {
                            first = (j_beg < ep.n_ctiles)
                                        ? (p.stream_meta[ep.stream_off + j_beg * kPagesPerTile] >> 8) : G;
                            last = (j_end > ep.n_ctiles)
                                       ? G : (p.stream_meta[ep.stream_off + j_end * kPagesPerTile - 1] >> 8);
                        }
                        if (slot_out)
                            for (int sl = 0; sl <= G; ++sl)
                                if (sl < first || sl > last) slot_out[sl] = kNegInf;
                        p.part_lse[rh] = lse;
                    }
                }
                if (!pair) *xinv = inv;
                // the row's final log-sum-exp (and the other split's part of the shared slot) for both halves: the
                // maximum exchange area is idle after the loop
                xmax_own[0] = pair ? pair_lse : lse;
                xmax_own[kXmaxPar] = pair_bnd;
            }
            if (ok) ok = pair_sync();                               // 1 / row sum (pair merge: the weight) reaches half B
        }
        // Masses: parked log-sums -> shares of the row's total, eight slots at a time (eight loads in flight; one
        // load, one exponential and one store per trip would pay a memory round trip per slot).  Without a peer the
        // owner does them while half B already writes its output channels and the last MMAs drain.  In a pair both
        // halves share them, after the output: the other CTA waits for that.  (Both orders were timed.)
        auto finish_masses = [&]() {
            if (!(row_valid && p.mass && !split_mode) || (!pair && !owner)) return;
            float *slots = p.mass + rh * p.mass_stride;
            const float *xref = owner ? xmax_own : xmax_other;      // written by the owner before the last pair sync
            const float ref = xref[0], extra = xref[kXmaxPar];
            int first = 0, last = G;
            if (pair) {                                             // the slots this CTA walked
                first = (j_beg < ep.n_ctiles) ? (p.stream_meta[ep.stream_off + j_beg * kPagesPerTile] >> 8) : G;
                last = (j_end > ep.n_ctiles) ? G : (p.stream_meta[ep.stream_off + j_end * kPagesPerTile - 1] >> 8);
            }
            for (int s0 = first + (pair ? 8 * hb : 0); s0 <= last; s0 += (pair ? 16 : 8)) {
                float v[8];
#pragma unroll
                for (int x = 0; x < 8; ++x) v[x] = (s0 + x <= last) ? slots[s0 + x] : kNegInf;
#pragma unroll
                for (int x = 0; x < 8; ++x) {
                    const int sl = s0 + x;
                    if (sl <= last && sl != skip_slot) {            // the shared slot is written by split 0 alone
                        float w = (ref != kNegInf) ? ex2(v[x] - ref) : 0.f;
                        if (sl == shared_slot && ref != kNegInf) w += ex2(extra - ref);
                        slots[sl] = w;
                    }
                }
            }
        };
        const bool masses_first = !pair;
        if (ok && masses_first) finish_masses();
        if (pair && !owner) w_peer = xmax_own[0];
        if (ok && n_tiles > 0 && !(pair && i != it.split)) {
            const float inv = *xinv;
            ok = mbar_wait(bar_o_done(i), 0, abort_flag, p.status);
            if (ok) {
                tc_fence_after();
                if constexpr (D == 128) {
                  if (pair) {
                    // This CTA finishes Q tile `it.split`: its own accumulator and what the peer sent (see the export
                    // above), each with its weight.  Thread (warp, lane) reads what thread (warp, lane) of the peer wrote.
                    const uint32_t peer = cluster_rank() ^ 1u;
                    const uint32_t ring_off = static_cast<uint32_t>(kQTiles * C::kTileBytes + (hb * 4 + q4) * 8192 + lane * 256);
                    if (i == it.split) {
                        uint8_t *stg = smem + i * C::kTileBytes + (hb * 4 + q4) * 4096;
#pragma unroll 1
                        for (int k = 0; k < 2 && ok; ++k) {         // 32 channels per pass
                            uint32_t o[32];
                            tmem_ld32_wait(t_o + static_cast<uint32_t>(hb * (D / 2) + k * 32), o);
                            if (k == 0) {
                                ok = mbar_wait<true>(bar_peer_o, 0, abort_flag, p.status);
                                // the peer may retire once its staging area has been read out: tell it
                                if (ok && hb == 0 && q4 == 0 && lane == 0) peer_arrive_relaxed(peer_addr(bar_peer_ack, peer));
                            }
                            if (!ok) break;
#pragma unroll
                            for (int cch = 0; cch < 4; ++cch) {
                                const float4 a = *reinterpret_cast<const float4 *>(smem + ring_off + (((k * 8 + 2 * cch) ^ (lane & 7)) << 4));
                                const float4 b = *reinterpret_cast<const float4 *>(smem + ring_off + (((k * 8 + 2 * cch + 1) ^ (lane & 7)) << 4));
                                auto mix = [&](uint32_t own, float theirs) { return fmaf(__uint_as_float(own), inv, theirs * w_peer); };
                                const __nv_bfloat162 b0 = __floats2bfloat162_rn(mix(o[8 * cch + 0], a.x), mix(o[8 * cch + 1], a.y));
                                const __nv_bfloat162 b1 = __floats2bfloat162_rn(mix(o[8 * cch + 2], a.z), mix(o[8 * cch + 3], a.w));
                                const __nv_bfloat162 b2 = __floats2bfloat162_rn(mix(o[8 * cch + 4], b.x), mix(o[8 * cch + 5], b.y));
                                const __nv_bfloat162 b3 = __floats2bfloat162_rn(mix(o[8 * cch + 6], b.z), mix(o[8 * cch + 7], b.w));
                                *reinterpret_cast<uint4 *>(stg + lane * 128 + (((k * 4 + cch) ^ (lane & 7)) << 4)) =
                                    make_uint4(*reinterpret_cast<const uint32_t *>(&b0), *reinterpret_cast<const uint32_t *>(&b1),
                                               *reinterpret_cast<const uint32_t *>(&b2), *reinterpret_cast<const uint32_t *>(&b3));
                            }
                        }
                        __syncwarp();
                        if (ok) {
#pragma unroll 1
                            for (int itr = 0; itr < 8; ++itr) {
                                const int rr = itr * 4 + (lane >> 3), cch = lane & 7;
                                const int r2 = q4 * 32 + rr;
                                const int t2 = it.t0 + i * tile_tokens + r2 / rep;
                                const long long rh2 = (static_cast<long long>(ep.q_off) + t2) * p.Hq + it.kvh * rep + r2 % rep;
                                const uint4 v = *reinterpret_cast<const uint4 *>(stg + rr * 128 + ((cch ^ (rr & 7)) << 4));
                                if (t2 < ep.n_q)
                                    *reinterpret_cast<uint4 *>(static_cast<__nv_bfloat16 *>(p.out) + rh2 * D + hb * (D / 2) + cch * 8) = v;
                            }
                        }
                    }
                  } else {
                    // Row-per-thread stores would touch 32 different rows per instruction.  Each warp stages its
                    // 32 rows x 128 bytes in the (now idle) shared memory of its Q tile, 16-byte chunks swizzled by
                    // row, and writes them out four whole 128-byte row pieces per instruction.
                    uint8_t *stg = smem + i * C::kTileBytes + (hb * 4 + q4) * 4096;
                    auto row_index = [&](int rr, bool &valid) -> long long {     // (row, head) index of staged row rr
                        const int r2 = q4 * 32 + rr;
                        const int t2 = it.t0 + i * tile_tokens + r2 / rep;
                        valid = t2 < ep.n_q;
                        const long long g2 = static_cast<long long>(ep.q_off) + t2;
                        return (split_mode ? (static_cast<long long>(it.split) * p.n_q_total + g2) : g2) * p.Hq +
                               it.kvh * rep + r2 % rep;
                    };
                    if (split_mode) {
#pragma unroll 1
                        for (int k = 0; k < 2; ++k) {               // 32 fp32 channels per pass
                            uint32_t o[32];
                            const int col = hb * (D / 2) + k * 32;
                            tmem_ld32_wait(t_o + static_cast<uint32_t>(col), o);
#pragma unroll
                            for (int cch = 0; cch < 8; ++cch)
                                *reinterpret_cast<float4 *>(stg + lane * 128 + ((cch ^ (lane & 7)) << 4)) =
                                    make_float4(__uint_as_float(o[4 * cch]) * inv, __uint_as_float(o[4 * cch + 1]) * inv,
                                                __uint_as_float(o[4 * cch + 2]) * inv, __uint_as_float(o[4 * cch + 3]) * inv);
                            __syncwarp();
#pragma unroll 1
                            for (int itr = 0; itr < 8; ++itr) {
                                const int rr = itr * 4 + (lane >> 3), cch = lane & 7;
                                bool valid;
                                const long long rh2 = row_index(rr, valid);
                                const float4 v = *reinterpret_cast<const float4 *>(stg + rr * 128 + ((cch ^ (rr & 7)) << 4));
                                if (valid) *reinterpret_cast<float4 *>(p.part_o + rh2 * D + col + cch * 4) = v;
                            }
                            __syncwarp();
                        }
                    } else {
#pragma unroll
                        for (int k = 0; k < 2; ++k) {               // 64 bf16 channels = 128 bytes per row
                            uint32_t o[32];
                            tmem_ld32_wait(t_o + static_cast<uint32_t>(hb * (D / 2) + k * 32), o);
#pragma unroll
                            for (int cch = 0; cch < 4; ++cch) {
                                uint32_t w[4];
#pragma unroll
                                for (int y = 0; y < 4; ++y) {
                                    const __nv_bfloat162 b = __floats2bfloat162_rn(
                                        __uint_as_float(o[8 * cch + 2 * y]) * inv, __uint_as_float(o[8 * cch + 2 * y + 1]) * inv);
                                    w[y] = *reinterpret_cast<const uint32_t *>(&b);
                                }
                                *reinterpret_cast<uint4 *>(stg + lane * 128 + (((k * 4 + cch) ^ (lane & 7)) << 4)) =
                                    make_uint4(w[0], w[1], w[2], w[3]);
                            }
                        }
                        __syncwarp();
#pragma unroll 1
                        for (int itr = 0; itr < 8; ++itr) {
                            const int rr = itr * 4 + (lane >> 3), cch = lane & 7;
                            bool valid;
                            const long long rh2 = row_index(rr, valid);
                            const uint4 v = *reinterpret_cast<const uint4 *>(stg + rr * 128 + ((cch ^ (rr & 7)) << 4));
                            if (valid)
                                *reinterpret_cast<uint4 *>(static_cast<__nv_bfloat16 *>(p.out) + rh2 * D + hb * (D / 2) + cch * 8) = v;
                        }
                    }
                  }
                } else {
#pragma unroll
                for (int k = 0; k < D / 64; ++k) {                  // this half's D/2 output channels
                    uint32_t o[32];
                    const int col = hb * (D / 2) + k * 32;
                    tmem_ld32_wait(t_o + static_cast<uint32_t>(col), o);
                    if (row_valid) {
                        if (split_mode) {
                            float4 *dst = reinterpret_cast<float4 *>(p.part_o + rh * D + col);
#pragma unroll
                            for (int x = 0; x < 8; ++x)
                                dst[x] = make_float4(__uint_as_float(o[4 * x]) * inv, __uint_as_float(o[4 * x + 1]) * inv,
                                                     __uint_as_float(o[4 * x + 2]) * inv, __uint_as_float(o[4 * x + 3]) * inv);
                        } else {
                            uint4 *dst = reinterpret_cast<uint4 *>(
                                static_cast<__nv_bfloat16 *>(p.out) + rh * D + col);
#pragma unroll
                            for (int x = 0; x < 4; ++x) {
                                uint32_t w[4];
#pragma unroll
                                for (int y = 0; y < 4; ++y) {
                                    const __nv_bfloat162 b = __floats2bfloat162_rn(
                                        __uint_as_float(o[8 * x + 2 * y]) * inv,
                                        __uint_as_float(o[8 * x + 2 * y + 1]) * inv);
                                    w[y] = *reinterpret_cast<const uint32_t *>(&b);
                                }
                                dst[x] = make_uint4(w[0], w[1], w[2], w[3]);
                            }
                        }
                    }
                }
                }
            }
        }
        if (ok && !masses_first) finish_masses();
        // what this CTA staged for its peer must have been fetched before the CTA may retire
        if (exported) ok = mbar_wait<true>(bar_peer_ack, 0, abort_flag, p.status);
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

#ifdef ENL_TRACE
extern "C" int enl_debug_trace(long long *out)
{
    return cudaMemcpyFromSymbol(out, g_trace, sizeof(g_trace)) == cudaSuccess ? 0 : -1;
}
#endif

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
