// Bidirectional attention rows with drift (Eq. 3, Eq. 4) as a STREAM over the key tiles: one CTA per
// (128 query rows, head) walks all keys twice, with the tensor core, the loads and the eight statistics warps
// overlapped through rings of operand tiles and two score accumulators in tensor memory.  bf16, head_dim 128,
// any number of keys.  For steps with many rows (block entries, long sequences, batches), where the kernel of
// attn_tc.cuh -- one tile per CTA, key ranges combined across a cluster -- spends its time in start-up and exchange.
//
//   pass 1   S_t = Q K_t^T for every key tile t (tcgen05.mma into accumulator t & 1); the statistics warps read
//            each S_t from tensor memory (lane = row, two threads per row) and keep a running maximum and sum:
//            the row's log-sum-exp
//   pass 2   S_t again (K comes back through the ring, from L2); p = 2^(t - lse), normalised BEFORE it is rounded
//            to bf16 (the rounding point of a plain implementation), the drift sum A = sum p (s - s_old) against the
//            stored row, the new stored row s, and P into shared memory as the A operand of O += P V_t (V as an
//            MN-major operand, accumulated in tensor memory over the tiles); S_{t+1} is computed while the
//            warps work on S_t
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

constexpr int THREADS = 320;              // warp 0: TMA, warp 1: MMA + tensor memory, warps 2..9: statistics / epilogue
constexpr int NK = 2, NV = 2;             // ring slots of K and V tiles
constexpr uint32_t TILE_BYTES = 2 * BOX_BYTES;       // [128][128] bf16 as two [128][64] boxes
constexpr uint32_t TMEM_COLS = 512;       // S0, S1, O (128 columns each)

__host__ __device__ constexpr size_t smem_bytes() { return (size_t)(2 + NK + NV) * TILE_BYTES + 1024; }     // Q, P, rings

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
    __shared__ uint64_t bars[4 + 2 * NK + 2 * NV + 4];
    __shared__ uint32_t tmem_base_sh;
    __shared__ int abort_sh;
    __shared__ float* prev_sh[ROWS];
    __shared__ float* lsep_sh[ROWS];
    __shared__ int valid_sh[ROWS];
    __shared__ float2 half_ml[2][ROWS];            // (maximum, sum) of each column half
    __shared__ float half_A[ROWS];                 // drift sum of the upper column half
    // Per statistics warp: a 32 x 16 block of stored-row values on its way between the layout tensor memory
    // imposes (lane = row) and the one global memory wants (four lanes = 64 contiguous bytes of a row); 16-byte
    // chunk c of row r sits at chunk c ^ ((r >> 1) & 3), which keeps both access patterns free of bank conflicts
    __shared__ float4 xpose[8][32 * 4];

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
    auto k_s = [&](int s) { return smem_base + (uint32_t)(2 + s) * TILE_BYTES; };
    auto v_s = [&](int s) { return smem_base + (uint32_t)(2 + NK + s) * TILE_BYTES; };
    const uint32_t bar_q = smem_u32(&bars[0]), bar_o = smem_u32(&bars[1]), bar_pfull = smem_u32(&bars[2]), bar_pfree = smem_u32(&bars[3]);
    auto bar_kfull = [&](int s) { return smem_u32(&bars[4 + s]); };
    auto bar_kfree = [&](int s) { return smem_u32(&bars[4 + NK + s]); };
    auto bar_vfull = [&](int s) { return smem_u32(&bars[4 + 2 * NK + s]); };
    auto bar_vfree = [&](int s) { return smem_u32(&bars[4 + 2 * NK + NV + s]); };
    auto bar_sfull = [&](int s) { return smem_u32(&bars[4 + 2 * NK + 2 * NV + s]); };
    auto bar_sfree = [&](int s) { return smem_u32(&bars[6 + 2 * NK + 2 * NV + s]); };

    if (threadIdx.x == 0) {
        mbar_init(bar_q, 1); mbar_init(bar_o, 1); mbar_init(bar_pfull, 8); mbar_init(bar_pfree, 1);
        for (int s = 0; s < NK; ++s) { mbar_init(bar_kfull(s), 1); mbar_init(bar_kfree(s), 1); }
        for (int s = 0; s < NV; ++s) { mbar_init(bar_vfull(s), 1); mbar_init(bar_vfree(s), 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(bar_sfull(s), 1); mbar_init(bar_sfree(s), 8); }
        abort_sh = 0;
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
    // K unit t (t < n: pass 1, else pass 2) holds key tile t mod n in ring slot t % NK; V unit j holds tile j in slot j % NV;
    // score accumulator of unit t: t & 1.  Use u of a ring slot (or accumulator) completes phase u & 1 of its barriers.

    if (warp == 0) {
        if (lane == 0) {
            auto clean = [&](int kt) {          // tile last written by an earlier forward: loadable before the dependency wait
                const int lo = kt * KEYS, hi = lo + KEYS;
                return hi <= a.dirty_lo || lo >= a.dirty_hi;
            };
            auto load_k = [&](int t) {
                const int s = t % NK, kt = t < n ? t : t - n;
                mbar_expect_tx(bar_kfull(s), TILE_BYTES);
                for (int kb = 0; kb < 2; ++kb)
                    tma_load_3d(k_s(s) + kb * BOX_BYTES, &map_k, bar_kfull(s), g_kv * DH + kb * 64, kt * KEYS, kv_seq);
            };
            auto load_v = [&](int j) {
                const int s = j % NV;
                mbar_expect_tx(bar_vfull(s), TILE_BYTES);
                for (int kb = 0; kb < 2; ++kb)
                    tma_load_3d(v_s(s) + kb * BOX_BYTES, &map_v, bar_vfull(s), g_kv * DH + kb * 64, j * KEYS, kv_seq);
            };
            int tk = 0, tv = 0;                 // K and V units requested so far
            bool ok = true;
            auto issue_k = [&]() {
                if (tk >= NK) ok = ok && mbar_wait(bar_kfree(tk % NK), (uint32_t)(tk / NK - 1) & 1u, abort_flag);
                if (ok) load_k(tk);
                ++tk;
            };
            auto issue_v = [&]() {
                if (tv >= NV) ok = ok && mbar_wait(bar_vfree(tv % NV), (uint32_t)(tv / NV - 1) & 1u, abort_flag);
                if (ok) load_v(tv);
                ++tv;
            };
            while (tk < min(NK, 2 * n) && clean(tk < n ? tk : tk - n)) issue_k();
            while (tv < min(NV, n) && clean(tv)) issue_v();
            pdl_wait();      // q, and the K / V rows written this step, come from the projection that ran just before
            trace_stamp(7);
            mbar_expect_tx(bar_q, TILE_BYTES);
            for (int kb = 0; kb < 2; ++kb) tma_load_2d(q_s + kb * BOX_BYTES, &map_q, bar_q, h * DH + kb * 64, row0);
            while (tk < n && ok) issue_k();
            while (tv < min(NV, n) && ok) issue_v();
            for (int j = 0; j < n && ok; ++j) {
                // K of pass-2 units j and j + 1 before the V tile whose slot only frees once P V_j has run (the MMA
                // warp issues S of unit j + 1 before P V_j)
                while (tk < min(2 * n, n + j + 2) && ok) issue_k();
                while (tv < min(n, j + NV + 1) && ok) issue_v();
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc_s = instr_desc_bf16(ROWS, KEYS);
            const uint32_t idesc_o = instr_desc_bf16(ROWS, DH) | (1u << 16);       // B (= V) is MN-major
            bool ok = mbar_wait(bar_q, 0, abort_flag);
            auto mma_s = [&](int t) {
                const int s = t % NK, b = t & 1;
                ok = ok && mbar_wait(bar_kfull(s), (uint32_t)(t / NK) & 1u, abort_flag);
                if (t >= 2) ok = ok && mbar_wait(bar_sfree(b), (uint32_t)((t >> 1) - 1) & 1u, abort_flag);
                if (!ok) return;
                tc_fence_after();
#pragma unroll
                for (int k = 0; k < DH / UMMA_K; ++k) {
                    const uint64_t da = smem_desc_sw128(q_s + (k >> 2) * BOX_BYTES) + (uint64_t)((k & 3) * 2);
                    const uint64_t db = smem_desc_sw128(k_s(s) + (k >> 2) * BOX_BYTES) + (uint64_t)((k & 3) * 2);
                    umma_bf16(tmem_base + (uint32_t)(b * KEYS), da, db, idesc_s, k > 0 ? 1u : 0u);
                }
                umma_commit(bar_kfree(s));
                umma_commit(bar_sfull(b));
            };
            for (int t = 0; t < n && ok; ++t) mma_s(t);
            if (ok) mma_s(n);
            for (int j = 0; j < n && ok; ++j) {
                if (j + 1 < n) mma_s(n + j + 1);
                const int s = j % NV;
                ok = ok && mbar_wait(bar_vfull(s), (uint32_t)(j / NV) & 1u, abort_flag) && mbar_wait(bar_pfull, (uint32_t)j & 1u, abort_flag);
                if (!ok) break;
                tc_fence_after();
#pragma unroll
                for (int k = 0; k < KEYS / UMMA_K; ++k) {
                    // A = P: K-major, 64 keys per 128-byte row;  B = V_j: 16 keys = two 8-row groups further down
                    const uint64_t da = smem_desc_sw128(p_s + (k >> 2) * BOX_BYTES) + (uint64_t)((k & 3) * 2);
                    const uint64_t db = smem_desc_mn_sw128(v_s(s) + (uint32_t)k * 2048u, BOX_BYTES);
                    umma_bf16(tmem_base + 2u * KEYS, da, db, idesc_o, (j > 0 || k > 0) ? 1u : 0u);
                }
                umma_commit(bar_vfree(s));
                umma_commit(bar_pfree);
            }
            umma_commit(bar_o);          // (also on failure: the statistics warps then see the abort flag)
        }
    } else {
        // ---- statistics / epilogue warps: TMEM lane = row; the two warps of a lane quarter split the columns ----
        const int ew = warp - 2;
        const int quarter = warp & 3;
        const int half = ew >> 2;
        const int row = quarter * 32 + lane;
        const uint32_t taddr0 = tmem_base + ((uint32_t)(quarter * 32) << 16);
        pdl_wait();            // the row table, q and the stored rows all come from earlier kernels of the stream
        if (half == 0) {
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
        }
        bar_sync_epi();
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
        if (half == 0 && lsep_sh[row] && a.record_kl) lse_old = __ldcg(lsep_sh[row]);
        const float scale2 = a.scale * LOG2E_F;
        bool ok = true;

        // ---- pass 1: running (maximum, sum) of this thread's columns ----
        float mx = -INFINITY, l = 0.f;
        for (int t = 0; t < n; ++t) {
            const int b = t & 1;
            ok = mbar_wait(bar_sfull(b), (uint32_t)(t >> 1) & 1u, abort_flag) && ok && !*abort_flag;
            ok = __all_sync(0xffffffffu, ok) != 0;
            if (!ok) break;
            tc_fence_after();
            if (use_old) {
                // pass 2 will want this tile's stored row: have it in L2 by then (two 128-byte lines per thread)
                const int kb = t * KEYS + half * 64;
                if (kb < a.N) asm volatile("prefetch.global.L2 [%0];" ::"l"(prev + kb));
                if (kb + 32 < a.N) asm volatile("prefetch.global.L2 [%0];" ::"l"(prev + kb + 32));
            }
            if (warp_valid) {
                uint32_t r[4][16];
#pragma unroll
                for (int u = 0; u < 4; ++u) tmem_ld16_issue(taddr0 + (uint32_t)(b * KEYS + half * 64 + 16 * u), r[u]);
                tmem_ld_wait();
                const int kb = t * KEYS + half * 64;
                float tm = -INFINITY;
#pragma unroll
                for (int u = 0; u < 4; ++u)
#pragma unroll
                    for (int i = 0; i < 16; ++i)
                        if (kb + 16 * u + i < a.N) tm = fmaxf(tm, __uint_as_float(r[u][i]));
                tm *= scale2;      // scale2 > 0: the maximum commutes with it
                const float nm = fmaxf(mx, tm);
                if (nm > -INFINITY) {
                    float sum = 0.f;
#pragma unroll
                    for (int u = 0; u < 4; ++u)
#pragma unroll
                        for (int i = 0; i < 16; ++i)
                            if (kb + 16 * u + i < a.N) sum += ex2(__uint_as_float(r[u][i]) * scale2 - nm);
                    l = l * ex2(mx - nm) + sum;       // (mx = -inf: l is 0 and 2^(-inf) = 0)
                }
                mx = nm;
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_sfree(b));
        }
        half_ml[half][row] = make_float2(mx, l);
        bar_sync_epi();
        float lse2;
        {
            const float2 h0 = half_ml[0][row], h1 = half_ml[1][row];
            const float M = fmaxf(h0.x, h1.x);
            float L = 0.f;
            if (h0.y > 0.f) L = fmaf(h0.y, ex2(h0.x - M), L);
            if (h1.y > 0.f) L = fmaf(h1.y, ex2(h1.x - M), L);
            lse2 = M + log2f(L);
        }
        float dlse = 0.f;
        if (half == 0) {
            // the row's log-sum-exp is kept in natural-log units, like the stored rows
            float* lsep = lsep_sh[row];
            const float lse = lse2 * LN2_F;
            dlse = lse - lse_old;
            if (lsep && valid && ok) *lsep = lse;
        }

        // ---- pass 2: probabilities (normalised before they are rounded to bf16), drift sum, the new stored row, P ----
        float A = 0.f;
        for (int j = 0; j < n && ok; ++j) {
            const int t = n + j, b = t & 1;
            const int kb = j * KEYS + half * 64;
            // The stored rows of this tile are requested before the wait for its scores.  Aligned rows (N % 4 == 0):
            // coalesced, lane -> (row 8 k + lane / 4, 16-byte chunk lane % 4) for k = 0..3 of every 16-column group u,
            // so that a warp instruction reads 64 contiguous bytes of each of eight rows; the values reach the lane
            // that owns the row through `xpose`.  Otherwise: each lane reads its own row, scalar.
            float oldv[64];              // coalesced layout [u][k][4], or (scalar path) the lane's own row
            if (vec && warp_old) {
#pragma unroll
                for (int u = 0; u < 4; ++u)
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const int rr = quarter * 32 + 8 * k + (lane >> 2);
                        const int col = kb + 16 * u + 4 * (lane & 3);
                        float4 o4 = make_float4(0.f, 0.f, 0.f, 0.f);
                        if (a.record_kl && prev_sh[rr] && col < a.N) o4 = __ldcg(reinterpret_cast<const float4*>(prev_sh[rr] + col));
                        oldv[16 * u + 4 * k] = o4.x; oldv[16 * u + 4 * k + 1] = o4.y; oldv[16 * u + 4 * k + 2] = o4.z; oldv[16 * u + 4 * k + 3] = o4.w;
                    }
            } else if (!vec && use_old) {
#pragma unroll
                for (int i = 0; i < 64; ++i) oldv[i] = (kb + i < a.N) ? __ldcg(prev + kb + i) : 0.f;
            }
            ok = mbar_wait(bar_sfull(b), (uint32_t)(t >> 1) & 1u, abort_flag) && ok && !*abort_flag;
            ok = __all_sync(0xffffffffu, ok) != 0;
            if (!ok) break;
            tc_fence_after();
            uint32_t pw[32];             // P of this thread's 64 columns, two bf16 per word
            if (warp_valid) {
                uint32_t r[4][16];
#pragma unroll
                for (int u = 0; u < 4; ++u) tmem_ld16_issue(taddr0 + (uint32_t)(b * KEYS + half * 64 + 16 * u), r[u]);
                tmem_ld_wait();
                float4* const xp = xpose[ew];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    float s_nat[16], pr[16], old16[16];
                    const int k16 = kb + 16 * u;
                    if (vec && warp_old) {
                        // coalesced layout -> the row's owner
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            const int lr = 8 * k + (lane >> 2);
                            xp[lr * 4 + ((lane & 3) ^ ((lr >> 1) & 3))] =
                                make_float4(oldv[16 * u + 4 * k], oldv[16 * u + 4 * k + 1], oldv[16 * u + 4 * k + 2], oldv[16 * u + 4 * k + 3]);
                        }
                        __syncwarp();
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            const float4 o4 = xp[lane * 4 + (c ^ ((lane >> 1) & 3))];
                            old16[4 * c] = o4.x; old16[4 * c + 1] = o4.y; old16[4 * c + 2] = o4.z; old16[4 * c + 3] = o4.w;
                        }
                        __syncwarp();
                    } else {
#pragma unroll
                        for (int i = 0; i < 16; ++i) old16[i] = (!vec && use_old) ? oldv[16 * u + i] : 0.f;
                    }
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const bool in = valid && (k16 + i < a.N);
                        const float tt = __uint_as_float(r[u][i]) * scale2;
                        const float p = in ? ex2(tt - lse2) : 0.f;     // rows that are not valid hand zeros to the tensor core
                        s_nat[i] = tt * LN2_F;
                        if (use_old && in) A = fmaf(p, s_nat[i] - old16[i], A);
                        pr[i] = p;
                    }
                    if (vec && warp_prev) {
                        // the new stored rows: the owner's values -> coalesced layout -> global memory
#pragma unroll
                        for (int c = 0; c < 4; ++c)
                            xp[lane * 4 + (c ^ ((lane >> 1) & 3))] = make_float4(s_nat[4 * c], s_nat[4 * c + 1], s_nat[4 * c + 2], s_nat[4 * c + 3]);
                        __syncwarp();
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            const int lr = 8 * k + (lane >> 2);
                            const int rr = quarter * 32 + lr;
                            const int col = k16 + 4 * (lane & 3);
                            if (prev_sh[rr] && valid_sh[rr] && col < a.N)
                                __stcg(reinterpret_cast<float4*>(prev_sh[rr] + col), xp[lr * 4 + ((lane & 3) ^ ((lr >> 1) & 3))]);
                        }
                        __syncwarp();
                    } else if (!vec && prev && valid) {
#pragma unroll
                        for (int i = 0; i < 16; ++i)
                            if (k16 + i < a.N) __stcg(prev + k16 + i, s_nat[i]);
                    }
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        __nv_bfloat162 bb = __floats2bfloat162_rn(pr[2 * i], pr[2 * i + 1]);
                        pw[8 * u + i] = *reinterpret_cast<uint32_t*>(&bb);
                    }
                }
            } else {
#pragma unroll
                for (int i = 0; i < 32; ++i) pw[i] = 0u;
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
            // P as the A operand of P V: row `row`, 16-byte chunks of its 128-byte row (64 keys), XOR-swizzled
            const uint32_t p_row = p_s + (uint32_t)half * BOX_BYTES + (uint32_t)row * 128u;
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const uint32_t dst = p_row + (uint32_t)((c ^ (row & 7)) << 4);
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(pw[4 * c]), "r"(pw[4 * c + 1]), "r"(pw[4 * c + 2]),
                             "r"(pw[4 * c + 3]) : "memory");
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_pfull);
        }

        // ---- output rows and drift ----
        if (half == 1) half_A[row] = A;
        ok = mbar_wait(bar_o, 0, abort_flag) && ok && !*abort_flag;
        ok = __all_sync(0xffffffffu, ok) != 0;
        tc_fence_after();
        bar_sync_epi();
        if (ok && warp_valid) {
            uint32_t r[4][16];
#pragma unroll
            for (int u = 0; u < 4; ++u) tmem_ld16_issue(taddr0 + 2u * KEYS + (uint32_t)(half * 64 + 16 * u), r[u]);
            tmem_ld_wait();
            if (valid && a.out) {
                __nv_bfloat16* dst = (__nv_bfloat16*)a.out + (size_t)(row0 + row) * dq + h * DH + half * 64;
#pragma unroll
                for (int u = 0; u < 4; ++u)
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
        if (ok && half == 0 && valid && a.kl)
            a.kl[(size_t)(row0 + row) * a.n_heads + h] = (lsep_sh[row] && a.record_kl) ? A + half_A[row] - dlse : 0.f;
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, TMEM_COLS);
    trace_stamp(312, 64);
    if (threadIdx.x == 0 && abort_sh && g.status) atomicExch(g.status, 1);
}

}  // namespace ast
}  // namespace ps
