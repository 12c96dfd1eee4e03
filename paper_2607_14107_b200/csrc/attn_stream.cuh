// Bidirectional attention rows with drift (Eq. 3, Eq. 4) as a STREAM over the key tiles: one CTA per
// (128 query rows, head) walks all keys twice, with the tensor core, the loads and the sixteen statistics warps
// overlapped through rings of operand tiles and two score accumulators in tensor memory.  bf16, head_dim 128,
// any number of keys.  For steps with many rows (block entries, long sequences, batches), where the kernel of
// attn_tc.cuh -- one tile per CTA, key ranges combined across a cluster -- spends its time in start-up and exchange.
//
//   pass 1   S_t = Q K_t^T for every key tile t (tcgen05.mma into accumulator t & 1); the statistics warps read
//            each S_t from tensor memory (lane = row, four threads per row) and keep a running maximum and sum:
//            the row's log-sum-exp
//   pass 2   S_t again (K comes back through the ring, from L2); p = 2^(t - lse), normalised BEFORE it is rounded
//            to bf16 (the rounding point of a plain implementation), the drift sum A = sum p (s - s_old) against the
//            stored row, the new stored row s, and P into shared memory as the A operand of O += P V_t (V as an
//            MN-major operand, accumulated in tensor memory over the tiles); S_{t+1} is computed while the
//            warps work on S_t
//   rows     the stored rows move as 512-byte bulk copies per row and tile between global memory and a staging tile
//            in shared memory: the statistics warps never wait on global memory
//   end      O from tensor memory to the output rows, KL = A - (lse - lse_old)
//
// Computing S twice costs tensor time (which this kernel has to spare) and saves the rescaling of a running
// output, the second rounding point it brings, and any exchange between CTAs.  Stored rows are scaled scores plus
// one log-sum-exp per row, as in attn_tc.cuh.  Every mbarrier wait is bounded.
#pragma once
#include "attn_tc.cuh"

namespace ps {
namespace ast {

using namespace atc;

constexpr int THREADS = 576;              // warp 0: TMA, warp 1: MMA + tensor memory, warps 2..17: statistics / epilogue
constexpr int NS = 2;                     // slots of the operand ring (K and V tiles in the order the tensor core uses them)
constexpr uint32_t XPITCH = 512 + 16;     // bytes per row of the stored-row staging tile (the pad spreads the rows over the banks)
constexpr uint32_t X_BYTES = ROWS * XPITCH;
constexpr uint32_t TILE_BYTES = 2 * BOX_BYTES;       // [128][128] bf16 as two [128][64] boxes
constexpr uint32_t TMEM_COLS = 512;       // S0, S1, O (128 columns each)

__host__ __device__ constexpr size_t smem_bytes() { return (size_t)(2 + NS) * TILE_BYTES + X_BYTES + 1024; }     // Q, P, ring, X

__device__ __forceinline__ void bar_sync_stat() { asm volatile("bar.sync 1, 512;" ::: "memory"); }
// one row segment global -> shared (bytes counted on the mbarrier) and shared -> global (bulk group); 16-byte aligned
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void bulk_store(void* dst, uint32_t src, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(src), "r"(bytes) : "memory");
}

struct Args {
    AttnArgs a;
    int rows_per_seq;       // forward rows per sequence (stand-alone: n_rows)
    int tiles_per_seq;      // 128-row tiles per sequence
    int* status;            // set to 1 when a bounded wait gave up (null: nowhere to report)
};

__global__ void __launch_bounds__(THREADS, 1)
attention_stream_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                        const __grid_constant__ CUtensorMap map_v, Args g) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bars[4 + 2 * NS + 4 + 2];
    __shared__ int cta_prev_sh;                    // any row of this CTA records
    __shared__ uint32_t tmem_base_sh;
    __shared__ int abort_sh;
    __shared__ float* prev_sh[ROWS];
    __shared__ float* lsep_sh[ROWS];
    __shared__ int valid_sh[ROWS];
    __shared__ float2 part_ml[4][ROWS];            // (maximum, sum) of each column quarter
    __shared__ float part_A[3][ROWS];              // drift sums of the upper three column quarters

    const AttnArgs& a = g.a;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int seq = blockIdx.x / g.tiles_per_seq, tile = blockIdx.x - seq * g.tiles_per_seq;
    const int h = blockIdx.y;
    const int g_kv = (h * a.n_kv) / a.n_heads;
    const int dq = a.n_heads * DH;
    const int row0 = seq * g.rows_per_seq + tile * ROWS;
    const int n_in_tile = min(ROWS, g.rows_per_seq - tile * ROWS);
    const int kv_seq = a.rows ? seq : 0;
    const int n = (a.N + KEYS - 1) / KEYS;                 // key tiles

    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t q_s = smem_base, p_s = smem_base + TILE_BYTES;
    auto ring_s = [&](int s) { return smem_base + (uint32_t)(2 + s) * TILE_BYTES; };
    const uint32_t bar_q = smem_u32(&bars[0]), bar_o = smem_u32(&bars[1]), bar_pfull = smem_u32(&bars[2]), bar_pfree = smem_u32(&bars[3]);
    auto bar_full = [&](int s) { return smem_u32(&bars[4 + s]); };
    auto bar_free = [&](int s) { return smem_u32(&bars[4 + NS + s]); };
    auto bar_sfull = [&](int s) { return smem_u32(&bars[4 + 2 * NS + s]); };
    auto bar_sfree = [&](int s) { return smem_u32(&bars[6 + 2 * NS + s]); };
    const uint32_t bar_x = smem_u32(&bars[8 + 2 * NS]), bar_w = smem_u32(&bars[9 + 2 * NS]);
    const uint32_t x_s = smem_base + (uint32_t)(2 + NS) * TILE_BYTES;

    if (threadIdx.x == 0) {
        mbar_init(bar_q, 1); mbar_init(bar_o, 1); mbar_init(bar_pfull, 16); mbar_init(bar_pfree, 1);
        for (int s = 0; s < NS; ++s) { mbar_init(bar_full(s), 1); mbar_init(bar_free(s), 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(bar_sfull(s), 1); mbar_init(bar_sfree(s), 16); }
        mbar_init(bar_x, ROWS);
        mbar_init(bar_w, 16);
        abort_sh = 0;
        cta_prev_sh = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32(&tmem_base_sh), TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    pdl_trigger();
    const uint32_t tmem_base = tmem_base_sh;
    volatile int* abort_flag = &abort_sh;
    // Operand units, in the order the tensor core consumes them (3 n in all, unit u in ring slot u % NS):
    //   K_0 .. K_{n-1}                          pass 1
    //   K_0, (K_1, V_0), (K_2, V_1), ..., V_{n-1}   pass 2: S of tile j + 1 is issued before P V of tile j
    // Score unit t (t < n: pass 1, else pass 2, tile t mod n) uses accumulator t & 1.  The k-th use of a ring slot or
    // accumulator completes phase k & 1 of its barriers.
    auto unit_tile = [&](int u, bool& is_v) {
        is_v = false;
        if (u < n) return u;
        if (u == n) return 0;
        const int w = u - n - 1;
        if (w == 2 * (n - 1)) { is_v = true; return n - 1; }
        if (w & 1) { is_v = true; return (w - 1) >> 1; }
        return (w >> 1) + 1;
    };

    if (warp == 0) {
        if (lane == 0) {
            auto clean = [&](int kt) {          // tile last written by an earlier forward: loadable before the dependency wait
                const int lo = kt * KEYS, hi = lo + KEYS;
                return hi <= a.dirty_lo || lo >= a.dirty_hi;
            };
            auto load = [&](int u) {
                bool is_v;
                const int kt = unit_tile(u, is_v), sl = u % NS;
                mbar_expect_tx(bar_full(sl), TILE_BYTES);
                for (int kb = 0; kb < 2; ++kb)
                    tma_load_3d(ring_s(sl) + kb * BOX_BYTES, is_v ? &map_v : &map_k, bar_full(sl), g_kv * DH + kb * 64, kt * KEYS, kv_seq);
            };
            int u = 0;
            bool ok = true;
            // the first ring slots need no wait; tiles that no kernel of this step writes are requested right away
            for (; u < min(NS, 3 * n); ++u) {
                bool is_v;
                if (!clean(unit_tile(u, is_v))) break;
                load(u);
            }
            pdl_wait();      // q, and the K / V rows written this step, come from the projection that ran just before
            trace_stamp(7);
            mbar_expect_tx(bar_q, TILE_BYTES);
            for (int kb = 0; kb < 2; ++kb) tma_load_2d(q_s + kb * BOX_BYTES, &map_q, bar_q, h * DH + kb * 64, row0);
            for (; u < 3 * n && ok; ++u) {
                if (u >= NS) ok = mbar_wait(bar_free(u % NS), (uint32_t)(u / NS - 1) & 1u, abort_flag);
                if (ok) load(u);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc_s = instr_desc_bf16(ROWS, KEYS);
            const uint32_t idesc_o = instr_desc_bf16(ROWS, DH) | (1u << 16);       // B (= V) is MN-major
            bool ok = mbar_wait(bar_q, 0, abort_flag);
            int u = 0;                   // operand units consumed so far
            auto take = [&]() {          // next unit of the ring: its slot, once the tile has landed
                const int sl = u % NS;
                ok = ok && mbar_wait(bar_full(sl), (uint32_t)(u / NS) & 1u, abort_flag);
                ++u;
                return sl;
            };
            auto mma_s = [&](int t) {
                const int sl = take(), b = t & 1;
                if (t >= 2) ok = ok && mbar_wait(bar_sfree(b), (uint32_t)((t >> 1) - 1) & 1u, abort_flag);
                if (!ok) return;
                tc_fence_after();
#pragma unroll
                for (int k = 0; k < DH / UMMA_K; ++k) {
                    const uint64_t da = smem_desc_sw128(q_s + (k >> 2) * BOX_BYTES) + (uint64_t)((k & 3) * 2);
                    const uint64_t db = smem_desc_sw128(ring_s(sl) + (k >> 2) * BOX_BYTES) + (uint64_t)((k & 3) * 2);
                    umma_bf16(tmem_base + (uint32_t)(b * KEYS), da, db, idesc_s, k > 0 ? 1u : 0u);
                }
                umma_commit(bar_free(sl));
                umma_commit(bar_sfull(b));
            };
            for (int t = 0; t < n && ok; ++t) mma_s(t);
            if (ok) mma_s(n);
            for (int j = 0; j < n && ok; ++j) {
                if (j + 1 < n) mma_s(n + j + 1);
                const int sl = take();
                ok = ok && mbar_wait(bar_pfull, (uint32_t)j & 1u, abort_flag);
                if (!ok) break;
                tc_fence_after();
#pragma unroll
                for (int k = 0; k < KEYS / UMMA_K; ++k) {
                    // A = P: K-major, 64 keys per 128-byte row;  B = V_j: 16 keys = two 8-row groups further down
                    const uint64_t da = smem_desc_sw128(p_s + (k >> 2) * BOX_BYTES) + (uint64_t)((k & 3) * 2);
                    const uint64_t db = smem_desc_mn_sw128(ring_s(sl) + (uint32_t)k * 2048u, BOX_BYTES);
                    umma_bf16(tmem_base + 2u * KEYS, da, db, idesc_o, (j > 0 || k > 0) ? 1u : 0u);
                }
                umma_commit(bar_free(sl));
                umma_commit(bar_pfree);
            }
            umma_commit(bar_o);          // (also on failure: the statistics warps then see the abort flag)
        }
    } else {
        // ---- statistics / epilogue warps: TMEM lane = row; the four warps of a lane quarter split the columns ----
        const int ew = warp - 2;
        const int quarter = warp & 3;             // tensor-memory lanes 32 * quarter .. + 31
        const int cq = ew >> 2;                   // columns 32 * cq .. + 31 of every tile
        const int row = quarter * 32 + lane;
        const uint32_t taddr0 = tmem_base + ((uint32_t)(quarter * 32) << 16);
        pdl_wait();            // the row table, q and the stored rows all come from earlier kernels of the stream
        if (cq == 0) {
            float* prev = nullptr; float* lsep = nullptr;
            int valid = 0;
            if (row < n_in_tile) {
                const int r = row0 + row;
                if (a.rows) {
                    const int4 rw = __ldg(reinterpret_cast<const int4*>(a.rows) + r);      // {seq, pos, widx, aidx}
                    if (rw.y >= 0) {
                        valid = 1;
                        if (a.cluster_K > 0 ? (row_is_proxy(rw.z) && a.pprev != nullptr) : (rw.z >= 0 && a.pprev != nullptr)) {
                            // recorded drift rows: the window rows, or (centroid proxies) the clusters' proxy rows
                            const size_t i = a.cluster_K > 0 ? ((size_t)rw.x * a.cluster_K + row_cluster(rw.z)) * a.n_heads + h
                                                             : ((size_t)rw.x * a.W_max + rw.z) * a.n_heads + h;
                            prev = a.pprev + i * a.N; lsep = a.pprev_lse + i;
                        } else if (rw.w >= 0 && a.aprev) {
                            const size_t i = ((size_t)rw.x * a.B + rw.w) * a.n_heads + h;
                            prev = a.aprev + i * a.N; lsep = a.aprev_lse + i;
                        }
                    }
                } else {
                    valid = 1;
                    if (a.pprev) { const size_t i = (size_t)r * a.n_heads + h; prev = a.pprev + i * a.N; lsep = a.pprev_lse + i; }
                }
            }
            prev_sh[row] = prev; lsep_sh[row] = lsep; valid_sh[row] = valid;
            if (prev) cta_prev_sh = 1;
        }
        bar_sync_stat();
        float* const prev = prev_sh[row];
        const bool valid = valid_sh[row] != 0;
        // tensor-memory loads are warp-wide (.sync.aligned): whether a warp reads at all is decided per warp
        const bool warp_valid = __any_sync(0xffffffffu, valid) != 0;
        const bool use_old = prev != nullptr && a.record_kl != 0;
        const bool vec = (a.N & 3) == 0;
        // stored rows are handled a warp at a time: nothing of it runs in a warp none of whose rows is recorded
        const bool warp_prev = __any_sync(0xffffffffu, prev != nullptr) != 0;
        const bool warp_old = warp_prev && a.record_kl != 0;
        float lse_old = 0.f;
        if (cq == 0 && lsep_sh[row] && a.record_kl) lse_old = __ldcg(lsep_sh[row]);
        const float scale2 = a.scale * LOG2E_F;
        bool ok = true;

        // ---- pass 1: running (maximum, sum) of this thread's columns (four independent chains each: two or four warps
        // per scheduler cannot hide one long dependent chain) ----
        float mx = -INFINITY, l = 0.f;
        for (int t = 0; t < n; ++t) {
            const int b = t & 1;
            ok = mbar_wait(bar_sfull(b), (uint32_t)(t >> 1) & 1u, abort_flag) && ok && !*abort_flag;
            ok = __all_sync(0xffffffffu, ok) != 0;
            if (!ok) break;
            tc_fence_after();
            const int kb = t * KEYS + cq * 32;
            if (use_old && vec && cq == 0 && (t & 3) == 0) {
                // pass 2 will want the stored row: bring it into L2 in pieces of four tiles (2 KB contiguous per row:
                // a DRAM page is opened for more than a sector or two)
                const int c0 = t * KEYS, nb = min(4 * KEYS, a.N - c0) * 4;
                asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(prev + c0), "r"(nb) : "memory");
            }
            if (warp_valid) {
                uint32_t r[2][16];
#pragma unroll
                for (int u = 0; u < 2; ++u) tmem_ld16_issue(taddr0 + (uint32_t)(b * KEYS + cq * 32 + 16 * u), r[u]);
                tmem_ld_wait();
                if (kb + 32 > a.N) {         // the tile's columns beyond the last key do not take part
#pragma unroll
                    for (int u = 0; u < 2; ++u)
#pragma unroll
                        for (int i = 0; i < 16; ++i)
                            if (kb + 16 * u + i >= a.N) r[u][i] = 0xff800000u;      // -inf
                }
                float tm4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
                for (int u = 0; u < 2; ++u)
#pragma unroll
                    for (int i = 0; i < 16; ++i) tm4[i & 3] = fmaxf(tm4[i & 3], __uint_as_float(r[u][i]));
                const float tm = fmaxf(fmaxf(tm4[0], tm4[1]), fmaxf(tm4[2], tm4[3])) * scale2;      // scale2 > 0: the maximum commutes with it
                const float nm = fmaxf(mx, tm);
                if (nm > -INFINITY) {
                    float s4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                    for (int u = 0; u < 2; ++u)
#pragma unroll
                        for (int i = 0; i < 16; ++i) s4[i & 3] += ex2(fmaf(__uint_as_float(r[u][i]), scale2, -nm));     // (2^-inf = 0)
                    l = l * ex2(mx - nm) + ((s4[0] + s4[1]) + (s4[2] + s4[3]));       // (mx = -inf: l is 0 and 2^(-inf) = 0)
                }
                mx = nm;
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_sfree(b));
        }
        part_ml[cq][row] = make_float2(mx, l);
        bar_sync_stat();
        float lse2;
        {
            float M = -INFINITY;
#pragma unroll
            for (int c = 0; c < 4; ++c) M = fmaxf(M, part_ml[c][row].x);
            float L = 0.f;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const float2 ml = part_ml[c][row];
                if (ml.y > 0.f) L = fmaf(ml.y, ex2(ml.x - M), L);
            }
            lse2 = M + log2f(L);
        }
        float dlse = 0.f;
        if (cq == 0) {
            // the row's log-sum-exp is kept in natural-log units, like the stored rows
            float* lsep = lsep_sh[row];
            const float lse = lse2 * LN2_F;
            dlse = lse - lse_old;
            if (lsep && valid && ok) *lsep = lse;
        }

        // ---- pass 2: probabilities (normalised before they are rounded to bf16), P, then drift sum and the new stored row ----
        // Stored rows travel as bulk copies between global memory and the staging tile X (one 512-byte segment per row
        // and tile, issued by the row's first thread): the statistics warps only ever touch shared memory, and DRAM
        // sees whole row segments.  "X is ready for tile j" is phase j of bar_x: the 128 issuing threads arrive on it
        // once the bulk store of tile j - 1 has read their row out of X, together with the bytes of the old row of
        // tile j when there is one.  Rows whose length is not a multiple of four floats (no 16-byte alignment) go the
        // plain way: every thread reads and writes its own row segment.
        float A4[4] = {0.f, 0.f, 0.f, 0.f};
        const float neg_lse2 = -lse2;
        const bool use_x = vec && cta_prev_sh != 0;              // (the same in every thread of the CTA)
        const uint32_t x_row = x_s + (uint32_t)row * XPITCH + (uint32_t)cq * 128u;
        auto x_ready = [&](int j) {         // row's first thread: X may take tile j; request the old row segment if there is one
            const int nb = min(KEYS, a.N - j * KEYS) * 4;
            if (use_old) {
                mbar_expect_tx(bar_x, (uint32_t)nb);
                bulk_load(x_s + (uint32_t)row * XPITCH, prev + j * KEYS, (uint32_t)nb, bar_x);
            } else {
                mbar_arrive(bar_x);
            }
        };
        if (use_x && cq == 0) x_ready(0);
        for (int j = 0; j < n && ok; ++j) {
            const int t = n + j, b = t & 1;
            const int kb = j * KEYS + cq * 32;
            const bool edge = kb + 32 > a.N;
            float oldv[32];              // plain path: the lane's own row segment
            if (!vec && use_old) {
#pragma unroll
                for (int i = 0; i < 32; ++i) oldv[i] = (kb + i < a.N) ? __ldcg(prev + kb + i) : 0.f;
            }
            ok = mbar_wait(bar_sfull(b), (uint32_t)(t >> 1) & 1u, abort_flag) && ok && !*abort_flag;
            ok = __all_sync(0xffffffffu, ok) != 0;
            if (!ok) break;
            tc_fence_after();
            uint32_t pw[16];             // P of this thread's 32 columns, two bf16 per word
            uint32_t r[2][16];
            float pr[32];
            if (warp_valid) {
#pragma unroll
                for (int u = 0; u < 2; ++u) tmem_ld16_issue(taddr0 + (uint32_t)(b * KEYS + cq * 32 + 16 * u), r[u]);
                tmem_ld_wait();
                if (edge || !valid) {        // columns beyond the last key, rows that are not valid: probability zero
#pragma unroll
                    for (int u = 0; u < 2; ++u)
#pragma unroll
                        for (int i = 0; i < 16; ++i)
                            if (!valid || kb + 16 * u + i >= a.N) r[u][i] = 0xff800000u;      // -inf
                }
#pragma unroll
                for (int i = 0; i < 32; ++i) pr[i] = ex2(fmaf(__uint_as_float(r[i >> 4][i & 15]), scale2, neg_lse2));      // (masked entries are -inf: p = 0)
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    __nv_bfloat162 bb = __floats2bfloat162_rn(pr[2 * i], pr[2 * i + 1]);
                    pw[i] = *reinterpret_cast<uint32_t*>(&bb);
                }
            } else {
#pragma unroll
                for (int i = 0; i < 16; ++i) pw[i] = 0u;
            }
            // the scores are in registers: the accumulator may take the tile after next
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_sfree(b));
            // P of the previous tile must have been consumed by its P V before the buffer is rewritten
            if (j > 0) {
                ok = mbar_wait(bar_pfree, (uint32_t)(j - 1) & 1u, abort_flag) && ok && !*abort_flag;
                ok = __all_sync(0xffffffffu, ok) != 0;
                if (!ok) break;
            }
            // P as the A operand of P V: row `row`, 16-byte chunks of its 128-byte row (64 keys per box), XOR-swizzled
            const uint32_t p_row = p_s + (uint32_t)(cq >> 1) * BOX_BYTES + (uint32_t)row * 128u;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const uint32_t dst = p_row + (uint32_t)((((cq & 1) * 4 + c) ^ (row & 7)) << 4);
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(pw[4 * c]), "r"(pw[4 * c + 1]), "r"(pw[4 * c + 2]),
                             "r"(pw[4 * c + 3]) : "memory");
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_pfull);
            // ---- the tensor core has what it needs; now the stored row of this tile
            if (use_x) {
                if (warp_prev) {
                    ok = mbar_wait(bar_x, (uint32_t)j & 1u, abort_flag) && ok && !*abort_flag;
                    ok = __all_sync(0xffffffffu, ok) != 0;
                    if (ok && warp_valid) {
#pragma unroll
                        for (int c = 0; c < 8; ++c) {
                            float o0, o1, o2, o3;
                            asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(o0), "=f"(o1), "=f"(o2), "=f"(o3) : "r"(x_row + 16u * c) : "memory");
                            float sn[4];
#pragma unroll
                            for (int i = 0; i < 4; ++i)       // (rounded products, never fused into the subtraction below: an unchanged row gives exactly zero)
                                sn[i] = __fmul_rn(__fmul_rn(__uint_as_float(r[c >> 2][4 * (c & 3) + i]), scale2), LN2_F);
                            if (use_old) {
                                const float od[4] = {o0, o1, o2, o3};
#pragma unroll
                                for (int i = 0; i < 4; ++i)
                                    if (pr[4 * c + i] > 0.f) A4[i] = fmaf(pr[4 * c + i], sn[i] - od[i], A4[i]);      // (p = 0: also the masked entries)
                            }
                            asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(x_row + 16u * c), "f"(sn[0]), "f"(sn[1]), "f"(sn[2]), "f"(sn[3]) : "memory");
                        }
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // the bulk store reads what was just written
                }
                // every row of X is complete once all sixteen warps have passed here (an mbarrier, not a named barrier:
                // its wait is bounded like every other)
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_w);
                if (cq == 0) {
                    ok = mbar_wait(bar_w, (uint32_t)j & 1u, abort_flag) && ok && !*abort_flag;
                    ok = __all_sync(0xffffffffu, ok) != 0;
                    if (!ok) break;
                    if (prev) {
                        const int nb = min(KEYS, a.N - j * KEYS) * 4;
                        bulk_store(prev + j * KEYS, x_s + (uint32_t)row * XPITCH, (uint32_t)nb);
                        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                        asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                    }
                    if (j + 1 < n) x_ready(j + 1);
                }
            } else if (warp_valid && prev && valid) {
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    const float sn = __fmul_rn(__fmul_rn(__uint_as_float(r[i >> 4][i & 15]), scale2), LN2_F);
                    if (use_old && pr[i] > 0.f) A4[i & 3] = fmaf(pr[i], sn - oldv[i], A4[i & 3]);
                    if (kb + i < a.N) __stcg(prev + kb + i, sn);
                }
            }
        }
        if (use_x && cq == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");      // the last stores have left

        // ---- output rows and drift ----
        const float A = (A4[0] + A4[1]) + (A4[2] + A4[3]);
        if (cq > 0) part_A[cq - 1][row] = A;
        ok = mbar_wait(bar_o, 0, abort_flag) && ok && !*abort_flag;
        ok = __all_sync(0xffffffffu, ok) != 0;
        tc_fence_after();
        bar_sync_stat();
        if (ok && warp_valid) {
            uint32_t r[2][16];
#pragma unroll
            for (int u = 0; u < 2; ++u) tmem_ld16_issue(taddr0 + 2u * KEYS + (uint32_t)(cq * 32 + 16 * u), r[u]);
            tmem_ld_wait();
            if (valid && a.out) {
                __nv_bfloat16* dst = (__nv_bfloat16*)a.out + (size_t)(row0 + row) * dq + h * DH + cq * 32;
#pragma unroll
                for (int u = 0; u < 2; ++u)
#pragma unroll
                    for (int c = 0; c < 2; ++c) {
                        uint32_t w[4];
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            __nv_bfloat162 bb = __floats2bfloat162_rn(__uint_as_float(r[u][8 * c + 2 * i]), __uint_as_float(r[u][8 * c + 2 * i + 1]));
                            w[i] = *reinterpret_cast<uint32_t*>(&bb);
                        }
                        *reinterpret_cast<uint4*>(dst + 16 * u + 8 * c) = make_uint4(w[0], w[1], w[2], w[3]);
                    }
            }
        }
        if (ok && cq == 0 && valid && a.kl)
            a.kl[(size_t)(row0 + row) * a.n_heads + h] =
                (lsep_sh[row] && a.record_kl) ? ((A + part_A[0][row]) + (part_A[1][row] + part_A[2][row])) - dlse : 0.f;
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, TMEM_COLS);
    trace_stamp(312, 64);
    if (threadIdx.x == 0 && abort_sh && g.status) atomicExch(g.status, 1);
}

}  // namespace ast
}  // namespace ps
