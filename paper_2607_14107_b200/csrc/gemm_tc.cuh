// Weight-streaming bf16 GEMM on 5th-generation tensor cores (tcgen05 + TMEM, operands staged by TMA).
//
//   out[m][n] = sum_k A[m][k] * W[n][k]      A: activations [M, K], W: weights [N_out, K]
//
// The decoding step multiplies a few dozen to a few hundred rows by every weight matrix, so the
// kernel is bound by streaming W from HBM.  Design points, each taken from a measurement:
//
//  * W is stored TILE-MAJOR: the 256 x 64 block (feature tile f, k block kb) is one contiguous
//    32 KB chunk at chunk index f * (K / 64) + kb, so a weight TMA is one sequential burst.
//    These loads carry the evict_first L2 policy when every weight byte is used once per launch
//    (a single token tile): a weight stream with the default policy pushed activations, partial tiles,
//    the K/V cache and instruction lines out of L2 (14 % of the decode time).
//  * One 128 x 256 x 16 MMA consumes 8 KB of weights and the tensor pipe issues one every ~150 ns at
//    the rate HBM delivers them, so the instruction shape is made as large as it gets: M = 128 tokens
//    x N = 256 features.  With the features on the small side of the instruction the tensor pipe, not
//    HBM, was the limit (~4 TB/s).  Rows beyond the live tokens are out-of-bounds rows of the
//    activation tensor map: TMA fills them with zeros without reading memory.
//  * Schedule.  Tile ids are rasterised (tile_ft) so that consecutive ids form a compact block of the
//    output.  With more tiles than CTAs, CTA c first takes the whole tiles c, c + G, ...: the grid
//    works on G consecutive ids at a time and operand tiles are shared through L2.  The remaining
//    tiles -- all of them in the decoding step, where there are fewer tiles than SMs -- are split
//    stream-K: the (tile, k block) units are dealt in equal contiguous ranges, so every SM streams the
//    same number of bytes whatever the matrix shape.  A range is a sequence of segments (one per
//    output tile touched).  A segment that covers its tile's whole K runs the epilogue straight from
//    tensor memory (two accumulators: the next segment's MMAs overlap it); a partial segment is
//    published to a workspace slot.
//  * Reduction of split tiles (one pass at the end, all 16 warps): once the contributors of a CTA's
//    partial tiles have published (arrival counters, bounded wait), the CTA adds the slots in
//    ascending-k order (deterministic, no floating-point atomics) for its share of the items
//    (one row x 16 columns; four columns when a tile has many contributors) and runs the epilogue.
//    Shares are balanced (a CTA with two partial tiles takes half a share of each); all of this
//    arithmetic (64-bit divisions) is done by an idle thread while the main loop runs.
//  * Programmatic dependent launch: weight tiles of the first pipeline stages are requested
//    before griddepcontrol.wait, i.e. while the previous kernel of the stream still drains;
//    activations, residuals and every global write come after it.
//
// Warp roles (512 threads): warp 0 = TMA producer, warp 1 = MMA issuer and TMEM owner,
// warps 2..5 = epilogue (TMEM lane quarter warp % 4 = 32 tokens each), warps 6..15 only take part in
// the reduction (its loads are pure L2 latency: more threads, fewer rounds).  Every mbarrier wait and
// every wait on a counter is bounded; on time-out the CTA raises a status word, stops issuing work and
// leaves in order.
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "kernels.cuh"

namespace ps {
namespace tc {

constexpr int BLOCK_T = 128;   // tokens per tile (UMMA M)
constexpr int BLOCK_F = 256;   // output features per tile (UMMA N)
constexpr int BLOCK_K = 64;    // bf16 elements per k block = one 128-byte swizzle row
constexpr int UMMA_K = 16;
constexpr int THREADS = 192;          // producer warp, MMA warp, four epilogue warps
// Launched block size: the warps beyond the six role warps sleep at a barrier until the fix-up pass, where the
// reduction of partial tiles is pure memory latency and more threads in flight mean fewer rounds.
constexpr int FIX_THREADS = 512;
constexpr int MAX_STAGES = 8;
constexpr uint32_t A_BYTES = BLOCK_T * BLOCK_K * 2;   // 16 KB
constexpr uint32_t W_BYTES = BLOCK_F * BLOCK_K * 2;   // 32 KB
constexpr uint32_t STAGE_BYTES = A_BYTES + W_BYTES;
constexpr long long WAIT_LIMIT_CYCLES = 4000000000LL;   // ~2 s

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok;
}
// Bounded wait.  Returns false when the limit ran out or another role already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (true) {
        for (int i = 0; i < 64; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > WAIT_LIMIT_CYCLES) { *abort_flag = 1; return false; }
    }
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y)
        : "memory");
}
// same with an L2 eviction policy: weights that are streamed once carry evict_first, so that they do not
// push activations, partial tiles, the K/V cache and instruction lines out of L2
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ void tma_load_2d_hint(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y, uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4}], [%2], %5;"
        ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "l"(policy)
        : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// ---- CTA pairs (cluster of two): one tcgen05.mma, issued by the even CTA, runs on both SMs' tensor cores -----------------
// address of the same shared-memory variable in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t mapa_u32(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// load into this CTA's shared memory; the bytes are counted on a barrier of either CTA of the pair
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar_cluster, int x, int y) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar_cluster), "r"(x), "r"(y)
        : "memory");
}
// D (256 x N, 128 rows in each CTA's tensor memory) += A (128 rows per CTA) x B (N / 2 rows per CTA); descriptors are
// the issuing CTA's, the peer's operands sit at the same shared-memory offsets
__device__ __forceinline__ void umma_bf16_pair(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n}\n"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// arrives on the barrier at this offset in both CTAs once the MMAs issued so far have completed
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"((uint16_t)3) : "memory");
}
// 16 consecutive accumulator columns of this thread's TMEM lane
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float* v) {
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
// the same load without the wait: several may be in flight before one tmem_ld_wait(); the registers may only
// be consumed by memory operations placed after the wait (its "memory" clobber orders them)
__device__ __forceinline__ void tmem_ld16_issue(uint32_t taddr, uint32_t* r) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
// the same wait for registers that arithmetic consumes: they are operands of the wait, so nothing that uses them moves above it
__device__ __forceinline__ void tmem_ld_wait16(uint32_t* r) {
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
                   "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15])
                 :: "memory");
}
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }

// Shared-memory matrix descriptor: K-major tile, rows of 128 bytes, 128-byte swizzle,
// 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)(1024u >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M x N.
__host__ __device__ inline uint32_t instr_desc_bf16(int m, int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

struct SkArgs {
    int M, N_out, K, stages;
    int tiles_f, tiles_t;
    float* partial;     // [2 * gridDim.x][tokens per CTA tile][BLOCK_F] fp32
    int* tile_counter;  // arrivals [tile] and, done_offset further on, finished shares [tile]; zero before
                        // launch, zero again after
    int done_offset;
    int* status;        // set to 1 on a wait time-out
    int w_stream;       // 1: every weight byte is read once by this launch: load it with the evict_first L2 policy
    int epi_groups;     // 1..3 groups of four warps drain an accumulator (groups beyond the first: warps 8-11, 12-15,
                        // which otherwise idle until the reduction pass); the 16-column chunks are dealt round-robin
    long long* trace;   // POLESTAR_TRACE builds: [gridDim.x][12] nanosecond stamps of this launch (null: off): 0 start,
                        // 1 set-up done, 2 dependencies resolved, 3 first stage full, 4 last MMA issued, 5 partial tiles
                        // published, 6 other contributors arrived, 8 share reduced, 7 end
};

__device__ __forceinline__ long long gtime() { long long t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)); return t; }
#ifdef POLESTAR_TRACE
#define SK_STAMP(i) do { if (g.trace) g.trace[(size_t)blockIdx.x * 12 + (i)] = gtime(); } while (0)
#else
#define SK_STAMP(i) do { } while (0)
#endif

// first unit of CTA c when U units are split over G CTAs
__device__ __forceinline__ long long sk_begin(long long U, int G, int c) { return (U * c) / G; }
__device__ __forceinline__ int sk_owner(long long U, int G, long long u) {
    int c = (int)((u * G) / U);
    while (c > 0 && sk_begin(U, G, c) > u) --c;
    while (c + 1 < G && sk_begin(U, G, c + 1) <= u) ++c;
    return c;
}

// Tile id -> (feature tile, token tile).  Ids run over chunks of RASTER_T token tiles: inside a chunk the token
// tile varies fastest, then the feature tile.  The G tiles that the CTAs work on at the same time (consecutive
// ids) then cover a compact block of the output, about sqrt(G) feature tiles x RASTER_T token tiles, so that
// every operand tile fetched into L2 is used by many CTAs while it is there.
constexpr int RASTER_T = 16;
__device__ __forceinline__ void tile_ft(int tile, int tiles_f, int tiles_t, int& f, int& t) {
    if (tiles_t <= RASTER_T) { f = tile / tiles_t; t = tile - f * tiles_t; return; }
    const int per_chunk = tiles_f * RASTER_T;
    const int chunk = tile / per_chunk;
    const int local = tile - chunk * per_chunk;
    const int tc = min(RASTER_T, tiles_t - chunk * RASTER_T);
    f = local / tc;
    t = chunk * RASTER_T + (local - f * tc);
}

// Number of partial tile segments in CTA c's unit range (0, 1 or 2): what it has to publish and then help reduce.
__device__ __forceinline__ int sk_partial_segments(long long U, int G, int c, int kb_total) {
    const long long b = sk_begin(U, G, c), e = sk_begin(U, G, c + 1);
    if (e <= b) return 0;
    const long long tb = b / kb_total, te = (e - 1) / kb_total;
    const bool head_cut = b != tb * kb_total, tail_cut = e != (te + 1) * kb_total;
    if (tb == te) return (head_cut || tail_cut) ? 1 : 0;
    return (head_cut ? 1 : 0) + (tail_cut ? 1 : 0);
}
__device__ __forceinline__ int ld_acquire_gpu(const int* p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Stale-row selection of the step (Sec. 4.1) riding on the O projection: eight of the warps of CTA 0 that are
// idle until the reduction pass do it while the weights stream (batch of one sequence, small window).
struct SelFuse {
    int on;
    StepDesc sd;
    StepSelArgs a;
};

// four fp32 values added onto dst in L2 (16-byte aligned)
__device__ __forceinline__ void red_add_v4(float* dst, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("red.relaxed.gpu.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(dst), "f"(__uint_as_float(a)), "f"(__uint_as_float(b)),
                 "f"(__uint_as_float(c)), "f"(__uint_as_float(d)) : "memory");
}

// TT = 128-row halves of a token tile.  TT = 2 (steps of several hundred rows, where the operands come from L2 and
// the tensor pipe is the limit): a CTA tile is 256 tokens x 256 features, two MMAs per k step share one weight tile, so
// a k block costs 64 KB of operands for twice the work of the 48 KB of TT = 1; both accumulators (2 x 256 columns) fill
// the tensor memory, so the epilogue of a segment no longer overlaps the next segment's MMAs.
//
// CG = 2 (with TT = 1; launched as clusters of two CTAs): a CTA pair works on a tile of 256 tokens x 256 features.  Each
// CTA loads its 128 tokens and HALF of the weight tile (128 features), the even CTA issues one MMA for both tensor cores
// (tcgen05.mma.cta_group::2, M = 256), and each CTA ends up with its 128 tokens x 256 features in its own tensor memory:
// 32 KB of operands per CTA and k block instead of 48, so six stages fit and the operand supply (bytes in flight against
// the load latency) no longer limits the MMA rate, while the two accumulators keep the epilogue overlapped.  The schedule
// treats the pair as one CTA (stream-K ranges, whole tiles first); everything after the MMAs (epilogue, partial tiles,
// reduction pass) is per CTA on its own 128 rows, with partial-tile slots and tile counters of its own.
template <typename T, int EPI, int TT = 1, int CG = 1>
__global__ void __launch_bounds__(FIX_THREADS, 1)
gemm_sk_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_a,
               SkArgs g, EpiArgs e, PostArgs post, SelFuse sf) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bars[2 * MAX_STAGES + 4];
    __shared__ uint32_t tmem_base_sh;
    __shared__ int abort_sh;
    __shared__ int last_sh;
    __shared__ int fx_par[2][8];          // per partial tile of this CTA: tile, c_lo, nseg, before, mine, w_all, tile_f, tile_t
    __shared__ int fx_n;
    __shared__ volatile int fx_ready;

    constexpr int BT = BLOCK_T * TT;                       // tokens per CTA tile
    constexpr uint32_t A_BYTES_T = A_BYTES * TT;           // activations of a stage: TT boxes of [128][64]
    constexpr uint32_t W_BYTES_C = W_BYTES / CG;           // weights of a stage in this CTA's shared memory
    constexpr uint32_t STAGE_T = A_BYTES_T + W_BYTES_C;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr bool PAIR = CG == 2;
    static_assert(!PAIR || TT == 1, "CTA pairs take 128-token halves");
    const int rank = PAIR ? (int)(blockIdx.x & 1u) : 0;                  // CTA within its pair (cluster of two along x)
    // scheduling unit: a CTA, or a CTA pair (both CTAs of a pair run the same schedule)
    const int G = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x, cta = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
    const int slot_cta = (int)blockIdx.x;                                // owner index of partial-tile slots
    if (threadIdx.x == 0) SK_STAMP(0);
    const int kb_total = g.K / BLOCK_K;
    // Schedule: with more tiles than CTAs, CTA c first takes the whole tiles c, c + G, c + 2G, ... (`dp` of them:
    // at any time the grid works on G consecutive tile ids, see tile_ft), and the last G + (tiles mod G) tiles
    // (or just the tiles mod G; all tiles, when there are fewer than G) are split stream-K: units (tile, k block) in contiguous ranges
    // [u_begin, u_end) per CTA, whose partial tiles are reduced in the fix-up pass.  U, u_begin, u_end and the
    // arithmetic derived from them count units of this stream-K part; its tiles have ids tile_base + u / kb_total.
    const int tiles_all = g.tiles_f * g.tiles_t;
    // (the stream-K part is the remainder r = tiles mod G when that leaves at most ~8 CTAs per tile, else G + r tiles)
    const int rem = tiles_all % G;
    const int dp = (tiles_all < G) ? 0 : ((rem == 0 || rem * 8 >= G) ? tiles_all / G : tiles_all / G - 1);
    const int tile_base = dp * G;
    const long long U = (long long)(tiles_all - tile_base) * kb_total;
    const long long u_begin = sk_begin(U, G, cta), u_end = sk_begin(U, G, cta + 1);
    const int n_tail = (int)(u_end - u_begin);
    const int n_units = dp * kb_total + n_tail;

    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t full0 = smem_u32(&bars[0]), empty0 = smem_u32(&bars[MAX_STAGES]);
    // two accumulators in tensor memory (segment s uses buffer s & 1): the epilogue of one segment
    // drains its buffer while the MMAs of the next segment already fill the other
    const uint32_t accum_full = smem_u32(&bars[2 * MAX_STAGES]), accum_empty = smem_u32(&bars[2 * MAX_STAGES + 2]);
    constexpr uint32_t ncols = 2 * BLOCK_F;

    if (threadIdx.x == 0) {
        for (int s = 0; s < g.stages; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
        for (int b2 = 0; b2 < 2; ++b2) {
            mbar_init(accum_full + 8 * b2, 1);
            mbar_init(accum_empty + 8 * b2, 4 * g.epi_groups * CG);      // one arrival per epilogue warp (of both CTAs)
        }
        abort_sh = 0;
        last_sh = 0;
        fx_ready = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32(&tmem_base_sh), ncols);
    tc_fence_before();
    if (PAIR) cluster_sync_all(); else __syncthreads();      // (pairs: the peer's barriers are initialised before anything arrives on them)
    tc_fence_after();
    pdl_trigger();
    if (threadIdx.x == 0) SK_STAMP(1);
    const uint32_t tmem_base = tmem_base_sh;
    volatile int* abort_flag = &abort_sh;

    if (threadIdx.x == THREADS) {
        // An idle thread works out, while the main loop runs, which partial tiles this CTA will help reduce and
        // which share of their items is its own (64-bit divisions that must not sit on the tail's critical path).
        // The partial tiles of the CTA's unit range follow from the range alone: its first tile if the range
        // starts inside it or ends before its end, and its last tile (when different) if the range ends inside it.
        // A tile's items (one row x 16 columns each) are dealt to its contributors in contiguous shares; a CTA that
        // contributes to two tiles takes half a share of each, so that every CTA reduces about as many items.
        int n_fix = 0;
        if (n_tail > 0 && !((EPI == EPI_RESID || EPI == EPI_DOWN) && e.accumulate)) {
            const long long tb = u_begin / kb_total, te = (u_end - 1) / kb_total;       // (stream-K part's own numbering)
            const bool head_cut = u_begin != tb * kb_total, tail_cut = u_end != (te + 1) * kb_total;
            int fix_tile[2] = {0, 0};
            if (tb == te) { if (head_cut || tail_cut) fix_tile[n_fix++] = (int)tb; }
            else {
                if (head_cut) fix_tile[n_fix++] = (int)tb;
                if (tail_cut) fix_tile[n_fix++] = (int)te;
            }
            for (int f = 0; f < n_fix; ++f) {
                const int tile = fix_tile[f];
                const long long tile_begin = (long long)tile * kb_total, tile_end = tile_begin + kb_total;
                const int c_lo = sk_owner(U, G, tile_begin), c_hi = sk_owner(U, G, tile_end - 1);
                const int nseg = c_hi - c_lo + 1;
                const int w_lo = sk_partial_segments(U, G, c_lo, kb_total) == 2 ? 1 : 2;
                const int w_hi = (nseg > 1 && sk_partial_segments(U, G, c_hi, kb_total) == 2) ? 1 : 2;
                fx_par[f][0] = tile_base + tile; fx_par[f][1] = c_lo; fx_par[f][2] = nseg;
                fx_par[f][3] = (cta == c_lo) ? 0 : w_lo + 2 * (cta - c_lo - 1);
                fx_par[f][4] = (cta == c_lo) ? w_lo : (cta == c_hi ? w_hi : 2);
                fx_par[f][5] = (nseg == 1) ? w_lo : w_lo + w_hi + 2 * (nseg - 2);
                tile_ft(tile_base + tile, g.tiles_f, g.tiles_t, fx_par[f][6], fx_par[f][7]);
            }
        }
        fx_n = n_fix;
        __threadfence_block();
        fx_ready = 1;
    }

    if constexpr (EPI == EPI_RESID) {
        if (sf.on && cta == 0 && warp >= 6 && warp < 14) {
            __shared__ float sel_dsh[SEL_SMALL_W];
            __shared__ int sel_flags[SEL_SMALL_W];
            __syncwarp();
            pdl_wait();                                  // the per-head drift comes from the attention kernel
            step_select_inline(sf.sd, sf.a, (int)threadIdx.x - THREADS, 256, 2, sel_dsh, sel_flags);
        }
    }

    if (warp == 0) {
        if (lane == 0) {
            // weights do not depend on the previous kernel: request the first stages right away
            const int pre = min(g.stages, n_units);
            const uint64_t pol = l2_policy_evict_first();
            // (tile, k block) of a unit are advanced incrementally: no 64-bit division per unit on this thread
            const int tail_tile0 = (int)(u_begin / kb_total), tail_kb0 = (int)(u_begin - (long long)tail_tile0 * kb_total);
            struct It { int j, tile, kb, f, t; };
            auto start = [&]() {
                It it;
                it.j = 0;
                if (dp > 0) { it.tile = cta; it.kb = 0; } else { it.tile = tile_base + tail_tile0; it.kb = tail_kb0; }
                tile_ft(it.tile, g.tiles_f, g.tiles_t, it.f, it.t);
                return it;
            };
            auto advance = [&](It& it) {
                if (++it.kb == kb_total) {
                    it.kb = 0;
                    ++it.j;
                    if (it.j < dp) it.tile = it.j * G + cta;
                    else if (it.j == dp && dp > 0) { it.tile = tile_base + tail_tile0; it.kb = tail_kb0; }
                    else ++it.tile;
                    tile_ft(it.tile, g.tiles_f, g.tiles_t, it.f, it.t);
                }
            };
            It iw = start();
            // pairs: the bytes of both CTAs' loads are counted on the even CTA's barrier, which alone expects them
            const uint32_t full_pair = PAIR ? mapa_u32(full0, 0) : 0u;
            for (int i = 0; i < pre; ++i, advance(iw)) {
                if (PAIR) {
                    if (rank == 0) mbar_expect_tx(full0 + 8 * i, 2 * STAGE_T);
                    tma_load_2d_pair(smem_base + i * STAGE_T + A_BYTES_T, &map_w, full_pair + 8 * i, 0,
                                     (iw.f * kb_total + iw.kb) * BLOCK_F + rank * (BLOCK_F / 2));
                    continue;
                }
                mbar_expect_tx(full0 + 8 * i, STAGE_T);
                if (g.w_stream) tma_load_2d_hint(smem_base + i * STAGE_T + A_BYTES_T, &map_w, full0 + 8 * i, 0,
                                                 (iw.f * kb_total + iw.kb) * BLOCK_F, pol);
                else tma_load_2d(smem_base + i * STAGE_T + A_BYTES_T, &map_w, full0 + 8 * i, 0, (iw.f * kb_total + iw.kb) * BLOCK_F);
            }
            pdl_wait();
            SK_STAMP(2);
            {
                It ia = start();
                for (int i = 0; i < pre; ++i, advance(ia)) {
                    if (PAIR) {
                        tma_load_2d_pair(smem_base + i * STAGE_T, &map_a, full_pair + 8 * i, ia.kb * BLOCK_K, (ia.t * CG + rank) * BT);
                        continue;
                    }
#pragma unroll
                    for (int hh = 0; hh < TT; ++hh)
                        tma_load_2d(smem_base + i * STAGE_T + hh * A_BYTES, &map_a, full0 + 8 * i, ia.kb * BLOCK_K, ia.t * BT + hh * BLOCK_T);
                }
            }
            for (int i = pre; i < n_units; ++i, advance(iw)) {
                const int s = i % g.stages;
                const uint32_t ph = (uint32_t)(i / g.stages) & 1u;
                if (!mbar_wait(empty0 + 8 * s, ph ^ 1u, abort_flag)) break;
                const uint32_t dst = smem_base + s * STAGE_T;
                if (PAIR) {
                    if (rank == 0) mbar_expect_tx(full0 + 8 * s, 2 * STAGE_T);
                    tma_load_2d_pair(dst + A_BYTES_T, &map_w, full_pair + 8 * s, 0, (iw.f * kb_total + iw.kb) * BLOCK_F + rank * (BLOCK_F / 2));
                    tma_load_2d_pair(dst, &map_a, full_pair + 8 * s, iw.kb * BLOCK_K, (iw.t * CG + rank) * BT);
                    continue;
                }
                mbar_expect_tx(full0 + 8 * s, STAGE_T);
                if (g.w_stream) tma_load_2d_hint(dst + A_BYTES_T, &map_w, full0 + 8 * s, 0, (iw.f * kb_total + iw.kb) * BLOCK_F, pol);
                else tma_load_2d(dst + A_BYTES_T, &map_w, full0 + 8 * s, 0, (iw.f * kb_total + iw.kb) * BLOCK_F);
#pragma unroll
                for (int hh = 0; hh < TT; ++hh)
                    tma_load_2d(dst + hh * A_BYTES, &map_a, full0 + 8 * s, iw.kb * BLOCK_K, iw.t * BT + hh * BLOCK_T);
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {
            const uint32_t idesc = instr_desc_bf16(BLOCK_T * CG, BLOCK_F);
            int seg = 0;
            bool seg_start = true;
            const int tail_kb0 = (int)(u_begin % kb_total);
            const int dp_units = dp * kb_total;
            int kb = dp > 0 ? 0 : tail_kb0;
            for (int i = 0; i < n_units; ++i, kb = (i == dp_units) ? tail_kb0 : ((kb + 1 == kb_total) ? 0 : kb + 1)) {
                const int s = i % g.stages;
                const uint32_t ph = (uint32_t)(i / g.stages) & 1u;
                if (TT == 1 && seg_start && seg > 1) {
                    // the epilogue must have drained this buffer's previous segment (seg - 2)
                    if (!mbar_wait(accum_empty + 8 * (seg & 1), (uint32_t)((seg >> 1) - 1) & 1u, abort_flag)) break;
                    tc_fence_after();
                }
                if (TT == 2 && seg_start && seg > 0) {
                    // one pair of accumulators: the epilogue must have drained the previous segment
                    if (!mbar_wait(accum_empty, (uint32_t)(seg - 1) & 1u, abort_flag)) break;
                    tc_fence_after();
                }
                if (!mbar_wait(full0 + 8 * s, ph, abort_flag)) break;
                if (i == 0) SK_STAMP(3);
                tc_fence_after();
                const uint32_t sa = smem_base + s * STAGE_T;
                const uint64_t dw = smem_desc_sw128(sa + A_BYTES_T);
#pragma unroll
                for (int k = 0; k < BLOCK_K / UMMA_K; ++k)
#pragma unroll
                    for (int hh = 0; hh < TT; ++hh) {
                        if (PAIR)
                            umma_bf16_pair(tmem_base + (uint32_t)((seg & 1) * BLOCK_F), smem_desc_sw128(sa) + (uint64_t)(k * 2),
                                           dw + (uint64_t)(k * 2), idesc, (!seg_start || k > 0) ? 1u : 0u);
                        else
                            umma_bf16(tmem_base + (uint32_t)((TT == 1 ? (seg & 1) : hh) * BLOCK_F), smem_desc_sw128(sa + hh * A_BYTES) + (uint64_t)(k * 2),
                                      dw + (uint64_t)(k * 2), idesc, (!seg_start || k > 0) ? 1u : 0u);
                    }
                if (PAIR) umma_commit_pair(empty0 + 8 * s); else umma_commit(empty0 + 8 * s);
                seg_start = false;
                if (kb == kb_total - 1 || i == n_units - 1) {
                    if (PAIR) umma_commit_pair(accum_full + 8 * (seg & 1)); else umma_commit(accum_full + (TT == 1 ? 8 * (seg & 1) : 0));
                    if (i == n_units - 1) SK_STAMP(4);
                    ++seg;
                    seg_start = true;
                }
            }
        }
    } else if (warp < 6 || (warp >= 8 && warp < 4 + 4 * g.epi_groups)) {
        // ---- epilogue warps: TMEM lane = token, column = feature ------------------------------------
        pdl_wait();
        trace_stamp(100 + EPI, 64);
        const int q = warp & 3;                      // a warp reaches the 32 lanes of its quarter only
        const int groups = g.epi_groups, gi = warp < 6 ? 0 : (warp - 4) >> 2;
        const int t_local = q * 32 + lane;
        const uint32_t taddr0 = tmem_base + ((uint32_t)(q * 32) << 16);
        const int Mv = e.m_count ? min(g.M, __ldg(e.m_count)) : g.M;
        int seg = 0;
        long long u = u_begin;
        for (int sgi = 0;; ++sgi) {
            int tile, k0, k1;
            if (sgi < dp) { tile = sgi * G + cta; k0 = 0; k1 = kb_total; }       // whole tiles first
            else {
                if (u >= u_end) break;
                const int lt = (int)(u / kb_total);
                k0 = (int)(u - (long long)lt * kb_total);
                const long long tile_end = (long long)(lt + 1) * kb_total;
                const long long seg_end = tile_end < u_end ? tile_end : u_end;
                k1 = (int)(seg_end - (long long)lt * kb_total);
                tile = tile_base + lt;
                u = seg_end;
            }
            int tile_f, tile_t;
            tile_ft(tile, g.tiles_f, g.tiles_t, tile_f, tile_t);
            const int n0 = tile_f * BLOCK_F;
            const bool whole = (k0 == 0 && k1 == kb_total);
            if (!mbar_wait(accum_full + (TT == 1 ? 8 * (seg & 1) : 0), (uint32_t)(TT == 1 ? (seg >> 1) : seg) & 1u, abort_flag)) break;
            tc_fence_after();
            const int which = (k0 == 0) ? 1 : 0;     // slot 0: my range starts inside this tile
#pragma unroll
            for (int hh = 0; hh < TT; ++hh) {
                const int m = (tile_t * CG + rank) * BT + hh * BLOCK_T + t_local;
                const bool live = m < Mv;
                const bool warp_live = (tile_t * CG + rank) * BT + hh * BLOCK_T + q * 32 < Mv;      // any live token in this warp's quarter
                const uint32_t taddr = taddr0 + (uint32_t)((TT == 1 ? (seg & 1) : hh) * BLOCK_F);
                if (whole) {
                    if (warp_live) {
                        // this warp's 16-column chunks of the half (dealt round-robin over the groups); the tensor-memory load
                        // of the next chunk is in flight during the epilogue of the current one
                        const int step = 16 * groups;
                        int c0 = 16 * (((gi - hh * (BLOCK_F / 16)) % groups + groups) % groups);
                        uint32_t ra[16], rb[16];
                        float v[16];
                        if (c0 < BLOCK_F) tmem_ld16_issue(taddr + (uint32_t)c0, ra);
                        while (c0 < BLOCK_F) {
                            const int c1 = c0 + step;
                            tmem_ld_wait16(ra);
                            if (c1 < BLOCK_F) tmem_ld16_issue(taddr + (uint32_t)c1, rb);
                            if (live) {
#pragma unroll
                                for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(ra[i]);
                                epilogue16<T, EPI>(e, m, n0 + c0, v);
                            }
                            if (c1 >= BLOCK_F) break;
                            c0 = c1 + step;
                            tmem_ld_wait16(rb);
                            if (c0 < BLOCK_F) tmem_ld16_issue(taddr + (uint32_t)c0, ra);
                            if (live) {
#pragma unroll
                                for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(rb[i]);
                                epilogue16<T, EPI>(e, m, n0 + c1, v);
                            }
                        }
                    }
                } else if ((EPI == EPI_RESID || EPI == EPI_DOWN) && e.accumulate) {
                    // partial segment of a projection whose output rows are the residual rows: add it onto them in L2
                    bool row_ok = live;
                    float* dst = e.out_f32 + (size_t)m * e.ld_out + n0;
                    if (EPI == EPI_DOWN && live) {
                        const int r0 = e.list ? __ldcg(e.list + m) : m;
                        const int4 rw = __ldg(reinterpret_cast<const int4*>(e.rows) + r0);       // {seq, pos, widx, aidx}
                        row_ok = rw.y >= 0;
                        dst = (e.within && rw.z >= 0) ? e.packet + ((size_t)rw.x * e.W_max + rw.z) * e.ld_out + n0
                                                      : e.out_f32 + (size_t)r0 * e.ld_out + n0;
                    }
                    if (warp_live) {
                        for (int c0 = 0; c0 < BLOCK_F; c0 += 64) {
                            if ((hh * (BLOCK_F / 64) + (c0 >> 6)) % groups != gi) continue;
                            uint32_t r[4][16];
#pragma unroll
                            for (int j = 0; j < 4; ++j) tmem_ld16_issue(taddr + (uint32_t)(c0 + 16 * j), r[j]);
                            tmem_ld_wait();
                            if (row_ok) {
#pragma unroll
                                for (int j = 0; j < 4; ++j)
#pragma unroll
                                    for (int c = 0; c < 16; c += 4)
                                        red_add_v4(dst + c0 + 16 * j + c, r[j][c], r[j][c + 1], r[j][c + 2], r[j][c + 3]);
                            }
                        }
                    }
                } else {
                    // partial segment: publish it now, reduce later (pass 2), so that publishing never
                    // waits on another CTA
                    float* part = g.partial + ((size_t)(2 * slot_cta + which) * BT + hh * BLOCK_T + t_local) * BLOCK_F;
                    if (warp_live) {
                        // 64 columns per round trip to TMEM (four loads in flight, one wait)
                        for (int c0 = 0; c0 < BLOCK_F; c0 += 64) {
                            if ((hh * (BLOCK_F / 64) + (c0 >> 6)) % groups != gi) continue;
                            uint32_t r[4][16];
#pragma unroll
                            for (int j = 0; j < 4; ++j) tmem_ld16_issue(taddr + (uint32_t)(c0 + 16 * j), r[j]);
                            tmem_ld_wait();
                            if (live) {
#pragma unroll
                                for (int j = 0; j < 4; ++j)
#pragma unroll
                                    for (int c = 0; c < 16; c += 4)
                                        *reinterpret_cast<uint4*>(part + c0 + 16 * j + c) = make_uint4(r[j][c], r[j][c + 1], r[j][c + 2], r[j][c + 3]);
                            }
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                if (PAIR) mbar_arrive_cluster(mapa_u32(accum_empty + 8 * (seg & 1), 0));      // the even CTA issues the MMAs
                else mbar_arrive(accum_empty + (TT == 1 ? 8 * (seg & 1) : 0));
            }
            if (!whole && !((EPI == EPI_RESID || EPI == EPI_DOWN) && e.accumulate)) {
                __threadfence();
                asm volatile("bar.sync 1, %0;" ::"r"(128 * groups) : "memory");
                if (threadIdx.x == 64) atomicAdd(&g.tile_counter[tile * CG + rank], 1);
            }
            ++seg;
        }
        if (threadIdx.x == 64) SK_STAMP(5);
    }

    // ---- pass 2 (all warps): every CTA that contributed to split tiles reduces its share of them ------------
    if (n_units > 0) {
        __syncwarp();
        pdl_wait();
        const int Mv = e.m_count ? min(g.M, __ldg(e.m_count)) : g.M;
        {
            const long long t0 = clock64();
            while (!fx_ready) { if (clock64() - t0 > WAIT_LIMIT_CYCLES) { *abort_flag = 1; break; } }
            __threadfence_block();
        }
        const int n_fix = fx_ready ? fx_n : 0;
        if (n_fix > 0) {
            // inside the CTA the items of both tiles form one list for all its threads
            int fix_tile[2] = {0, 0}, f_lo[2] = {0, 0}, f_n[2] = {0, 0}, f_clo[2] = {0, 0}, f_nseg[2] = {1, 1};
            int f_tf[2] = {0, 0}, f_tt[2] = {0, 0};
#pragma unroll
            for (int f = 0; f < 2; ++f) {
                if (f < n_fix) {
                    fix_tile[f] = fx_par[f][0]; f_clo[f] = fx_par[f][1]; f_nseg[f] = fx_par[f][2];
                    const int before = fx_par[f][3], mine = fx_par[f][4], w_all = fx_par[f][5];
                    f_tf[f] = fx_par[f][6]; f_tt[f] = fx_par[f][7];
                    const int tile_t = f_tt[f];
                    const int n_live = max(0, min(BT, Mv - (tile_t * CG + rank) * BT));
                    const int n_items = n_live * (BLOCK_F / 16);
                    f_lo[f] = (n_items * before) / w_all;
                    f_n[f] = (n_items * (before + mine)) / w_all - f_lo[f];
                }
            }
            const int total = f_n[0] + f_n[1];
            if ((int)threadIdx.x < total) {
                // pull what the epilogue of this thread's first item reads into L1 while the tiles are still arriving
                const int f = (int)threadIdx.x < f_n[0] ? 0 : 1;
                const int item = f_lo[f] + (int)threadIdx.x - (f ? f_n[0] : 0);
                const int tile = fix_tile[f];
                epilogue_prefetch<T, EPI>(e, (f_tt[f] * CG + rank) * BT + item / (BLOCK_F / 16), f_tf[f] * BLOCK_F + (item % (BLOCK_F / 16)) * 16);
            }
            if (threadIdx.x == 64) {
                // bounded wait until all contributors have published their partial tiles
                const long long t0 = clock64();
                int ok = 1;
                for (int f = 0; f < n_fix && ok; ++f) {
                    while (ld_acquire_gpu(&g.tile_counter[fix_tile[f] * CG + rank]) < f_nseg[f]) {
                        if (*abort_flag || clock64() - t0 > WAIT_LIMIT_CYCLES) { ok = 0; *abort_flag = 1; break; }
                        __nanosleep(64);
                    }
                }
                last_sh = ok;
                SK_STAMP(6);
            }
            __syncthreads();
            if ((EPI == EPI_RESID || EPI == EPI_DOWN) && last_sh && max(f_nseg[0], f_nseg[1]) > 4) {
                // Many contributors per tile (few output tiles): four threads share an item, each owning four
                // columns, so that one float4 per contributor is in flight for all contributors at once (one
                // round trip to L2 instead of one per group of four contributors).  Same summation order.
                for (int i4 = (int)threadIdx.x; i4 < 4 * total; i4 += FIX_THREADS) {
                    const int i = i4 >> 2;
                    const int f = i < f_n[0] ? 0 : 1;
                    const int item = f_lo[f] + i - (f ? f_n[0] : 0);
                    const int tile = fix_tile[f];
                    const int c_lo = f_clo[f], nseg = f_nseg[f];
                    const int tl = item / (BLOCK_F / 16), c0 = (item % (BLOCK_F / 16)) * 16 + (i4 & 3) * 4;
                    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
                    for (int sg0 = 0; sg0 < nseg; sg0 += 16) {
                        float4 tv[16];
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            const int cc = c_lo + sg0 + j;
                            const int wsl = (cc == c_lo) ? 1 : 0;
                            tv[j] = (sg0 + j < nseg)
                                        ? __ldcg(reinterpret_cast<const float4*>(g.partial + ((size_t)(2 * (cc * CG + rank) + wsl) * BT + tl) * BLOCK_F + c0))
                                        : make_float4(0.f, 0.f, 0.f, 0.f);
                        }
#pragma unroll
                        for (int j = 0; j < 16; ++j) { acc.x += tv[j].x; acc.y += tv[j].y; acc.z += tv[j].z; acc.w += tv[j].w; }
                    }
                    epilogue4<T, EPI>(e, (f_tt[f] * CG + rank) * BT + tl, f_tf[f] * BLOCK_F + c0, acc);
                }
            } else if (last_sh) {
                for (int i = (int)threadIdx.x; i < total; i += FIX_THREADS) {
                    const int f = i < f_n[0] ? 0 : 1;
                    const int item = f_lo[f] + i - (f ? f_n[0] : 0);
                    const int tile = fix_tile[f];
                    const int c_lo = f_clo[f], nseg = f_nseg[f];
                    const int tl = item / (BLOCK_F / 16), c0 = (item % (BLOCK_F / 16)) * 16;
                    float acc[16];
#pragma unroll
                    for (int x = 0; x < 16; ++x) acc[x] = 0.f;
                    for (int sg0 = 0; sg0 < nseg; sg0 += 4) {
                        float4 tv[4][4];
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const int cc = c_lo + sg0 + j;
                            if (sg0 + j < nseg) {
                                // a CTA whose range starts inside the tile wrote slot 0, otherwise slot 1
                                // (only the tile's first contributor can start at or before the tile's first unit)
                                const int wsl = (cc == c_lo) ? 1 : 0;
                                const float4* ps = reinterpret_cast<const float4*>(
                                    g.partial + ((size_t)(2 * (cc * CG + rank) + wsl) * BT + tl) * BLOCK_F + c0);
#pragma unroll
                                for (int x = 0; x < 4; ++x) tv[j][x] = __ldcg(ps + x);
                            } else {
#pragma unroll
                                for (int x = 0; x < 4; ++x) tv[j][x] = make_float4(0.f, 0.f, 0.f, 0.f);
                            }
                        }
#pragma unroll
                        for (int j = 0; j < 4; ++j)
#pragma unroll
                            for (int x = 0; x < 4; ++x) {
                                acc[4 * x] += tv[j][x].x; acc[4 * x + 1] += tv[j][x].y;
                                acc[4 * x + 2] += tv[j][x].z; acc[4 * x + 3] += tv[j][x].w;
                            }
                    }
                    const int mm = (f_tt[f] * CG + rank) * BT + tl;
                    const int n0 = f_tf[f] * BLOCK_F;
                    epilogue16<T, EPI>(e, mm, n0 + c0, acc);
                }
            }
            if (threadIdx.x == 64) SK_STAMP(8);
            __syncthreads();
            if (threadIdx.x == 64 && last_sh) {
                // the last contributor to finish its share re-arms the tile's counters for the next launch
                for (int f = 0; f < n_fix; ++f) {
                    const int tile = fix_tile[f] * CG + rank;
                    const int prev = atomicAdd(&g.tile_counter[g.done_offset + tile], 1);
                    if (prev == f_nseg[f] - 1) { g.tile_counter[tile] = 0; g.tile_counter[g.done_offset + tile] = 0; }
                }
            }
        }
    }

    tc_fence_before();
    // (pairs: neither CTA leaves while the other may still arrive on its barriers or its MMAs read this shared memory)
    if (PAIR) cluster_sync_all(); else __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, ncols);
    if constexpr (EPI == EPI_RESID || EPI == EPI_DOWN) {
        if (post.kind != 0) {
            // Every output store of this CTA is issued (barrier above).  Add to the grid's counter, wait until
            // all CTAs have done so (all are resident: the grid has at most one CTA per SM), then share out the rows.
            __shared__ float post_red[33];
            __shared__ int post_ok;
            if (threadIdx.x == 0) { __threadfence(); atomicAdd(post.counter, 1u); }
            if ((int)blockIdx.x < post.n_rows) {
                if (threadIdx.x == 0) {
                    const long long t0 = clock64();
                    int ok = 1;
                    while ((int)((unsigned)ld_acquire_gpu(reinterpret_cast<const int*>(post.counter)) - post.expect) < 0) {
                        if (*abort_flag || clock64() - t0 > WAIT_LIMIT_CYCLES) { ok = 0; *abort_flag = 1; break; }
                        __nanosleep(32);
                    }
                    post_ok = ok;
                }
                __syncthreads();
                if (post_ok) {
                    for (int r = (int)blockIdx.x; r < post.n_rows; r += (int)gridDim.x) {
                        if (post.kind == 1)
                            prep_rows_row<T>(r, post.x, post.list, post.m_count, post.gain, post.eps, post.d, (T*)post.a_out, post_red,
                                             post.rows, const_cast<float*>(post.packet), post.sd.W_max);
                        else
                            prep_qkv_row<T>(post.sd, r, post.rows, post.x, post.hc, post.packet, post.patch, post.gain, post.eps,
                                            post.d, (T*)post.a_out, post.kvflag, post_red, post.ct);
                    }
                }
            }
        }
    }
    if (threadIdx.x == 0) SK_STAMP(7);
    trace_stamp(200 + EPI, 0);
    if (threadIdx.x == 0 && abort_sh) atomicExch(g.status, 1);
}

}  // namespace tc
}  // namespace ps
