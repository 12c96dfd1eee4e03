// A chain of weight-streaming GEMMs of one decoding step in ONE persistent kernel (O projection -> RMSNorm ->
// gate/up -> down -> patch + RMSNorm -> the next layer's QKV projection).  Each of these projections multiplies at most 128 rows by its weights, so every one of them is
// a stream-K launch of gemm_sk_kernel whose weight stream takes 4-27 us and whose drain, partial-tile exchange and
// kernel boundary take another ~10 us.  Chained, the boundary becomes a grid-wide counter, and while one
// projection drains and reduces, the TMA producer already fills the operand ring with the next projection's
// weights (they depend on nothing), so the next main loop starts with a full ring.  Measured on the 8B shape:
// 4 us per layer less than three launches plus the RMSNorm kernel (the grid-wide counter costs about what a
// kernel boundary costs; the gain is the ring filled ahead and one launch instead of four).
//
// Restrictions (the decoding regime): one token tile per projection (M <= 128), no more output tiles than CTAs.
// Every projection keeps the stream-K grid it would have alone (ChainProb::G); the launch has the largest of them.  Everything else -- tile-major weights with the evict_first
// policy, tcgen05 128 x 256 x 16 MMAs into two TMEM accumulators, published partial tiles reduced in ascending-k
// order by all 16 warps -- is as in gemm_tc.cuh, whose helpers this file uses.  All CTAs of the grid are resident
// (at most one per SM), so the grid-wide counters cannot deadlock; their waits are bounded all the same.
#pragma once
#include "gemm_tc.cuh"

namespace ps {
namespace tc {

constexpr int CHAIN_MAX = 4;

struct ChainProb {
    int M, N_out, K, tiles_f;     // one token tile; tiles_f = N_out / 256 output tiles
    int G;                        // CTAs that work on this projection (the first G of the grid; the rest only take part
                                  // in the grid-wide counters and the row staging)
    int epi;                      // EPI_RESID, EPI_SWIGLU, EPI_DOWN or EPI_QKV
    int norm_after;               // row staging between this projection and the next (post): 1 RMSNorm of the output
                                  // rows, 2 patch + RMSNorm of the next layer's QKV input (Algorithm 1 "Patch")
    EpiArgs e;
    PostArgs post;
};
struct ChainArgs {
    int n, stages;
    float* partial;
    int* tile_counter;
    int done_offset;
    int* status;
    unsigned* bar_counter;        // grid-wide arrival counter, never reset
    unsigned bar_base;            // its value when this launch starts: barrier k is passed at bar_base + (k + 1) * G
    ChainProb p[CHAIN_MAX];
};
struct ChainMaps {
    CUtensorMap w[CHAIN_MAX];
    CUtensorMap a[CHAIN_MAX];
};

template <typename T>
__device__ __forceinline__ void epi16_dyn(int kind, const EpiArgs& e, int m, int n, const float* v) {
    if (kind == EPI_RESID) epilogue16<T, EPI_RESID>(e, m, n, v);
    else if (kind == EPI_SWIGLU) epilogue16<T, EPI_SWIGLU>(e, m, n, v);
    else if (kind == EPI_DOWN) epilogue16<T, EPI_DOWN>(e, m, n, v);
    else epilogue16<T, EPI_QKV>(e, m, n, v);
}
template <typename T>
__device__ __forceinline__ void epi4_dyn(int kind, const EpiArgs& e, int m, int n, float4 v) {
    if (kind == EPI_RESID) epilogue4<T, EPI_RESID>(e, m, n, v);
    else epilogue4<T, EPI_DOWN>(e, m, n, v);
}
__device__ __forceinline__ void fence_async_global() { asm volatile("fence.proxy.async.global;" ::: "memory"); }


// One word counts the arrivals of the whole grid (spreading it over several words made every poll several
// dependent acquire loads and was slower).
__device__ __forceinline__ void grid_counter_arrive(unsigned* counter, int cta) {
    (void)cta;
    atomicAdd(counter, 1u);
}
// one thread: wait until the grid-wide counter has reached `expect` (wrap-safe), bounded
__device__ __forceinline__ bool grid_counter_wait(const unsigned* counter, unsigned expect, volatile int* abort_flag,
                                                  long long limit_cycles = WAIT_LIMIT_CYCLES) {
    const long long t0 = clock64();
    while ((int)((unsigned)ld_acquire_gpu(reinterpret_cast<const int*>(counter)) - expect) < 0) {
        if (*abort_flag || clock64() - t0 > limit_cycles) { *abort_flag = 1; return false; }
        __nanosleep(32);
    }
    return true;
}

// The bounded wait on its own: one thread waits until *counter reaches `expect` or `limit_cycles` have passed, and
// reports which (status 1 = gave up).  No TMA, no mbarrier, nothing else in flight: what a caller uses to check that a
// wait nobody satisfies ends in an error code and leaves the context usable.
__global__ void wait_probe_kernel(const unsigned* counter, unsigned expect, long long limit_cycles, int* status) {
    __shared__ int abort_sh;
    abort_sh = 0;
    const bool ok = grid_counter_wait(counter, expect, &abort_sh, limit_cycles);
    *status = ok ? 0 : 1;
}

template <typename T>
__global__ void __launch_bounds__(FIX_THREADS, 1)
gemm_chain_kernel(const __grid_constant__ ChainMaps maps, const __grid_constant__ ChainArgs ca, SelFuse sf) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bars[2 * MAX_STAGES + 4];
    __shared__ uint32_t tmem_base_sh;
    __shared__ int abort_sh;
    __shared__ int last_sh;
    __shared__ int fx_par[CHAIN_MAX][2][8];   // per projection and partial tile: tile, c_lo, nseg, before, mine, w_all
    __shared__ int fx_n[CHAIN_MAX];
    __shared__ volatile int fx_ready;
    __shared__ float post_red[33];
    __shared__ int post_ok;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = gridDim.x, cta = blockIdx.x;
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t full0 = smem_u32(&bars[0]), empty0 = smem_u32(&bars[MAX_STAGES]);
    const uint32_t accum_full = smem_u32(&bars[2 * MAX_STAGES]), accum_empty = smem_u32(&bars[2 * MAX_STAGES + 2]);
    constexpr uint32_t ncols = 2 * BLOCK_F;
    const int stages = ca.stages;

    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
        for (int b2 = 0; b2 < 2; ++b2) {
            mbar_init(accum_full + 8 * b2, 1);
            mbar_init(accum_empty + 8 * b2, 4);
        }
        abort_sh = 0;
        last_sh = 0;
        fx_ready = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32(&tmem_base_sh), ncols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    pdl_trigger();
    const uint32_t tmem_base = tmem_base_sh;
    volatile int* abort_flag = &abort_sh;

    // unit range of this CTA in projection p (units = (output tile, k block), dealt in equal contiguous ranges)
    auto range = [&](int p, int& kb_total, long long& U, long long& u_begin, long long& u_end) {
        kb_total = ca.p[p].K / BLOCK_K;
        U = (long long)ca.p[p].tiles_f * kb_total;
        const int Gp = ca.p[p].G;
        u_begin = cta < Gp ? sk_begin(U, Gp, cta) : 0;
        u_end = cta < Gp ? sk_begin(U, Gp, cta + 1) : 0;
    };

    if (threadIdx.x == THREADS) {
        // an idle thread works out, for every projection, which partial tiles this CTA helps reduce and its share
        for (int p = 0; p < ca.n; ++p) {
            int kb_total; long long U, u_begin, u_end;
            range(p, kb_total, U, u_begin, u_end);
            const int Gp = ca.p[p].G;
            int n_fix = 0;
            if (u_end > u_begin && !ca.p[p].e.accumulate) {
                const long long tb = u_begin / kb_total, te = (u_end - 1) / kb_total;
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
                    const int c_lo = sk_owner(U, Gp, tile_begin), c_hi = sk_owner(U, Gp, tile_end - 1);
                    const int nseg = c_hi - c_lo + 1;
                    const int w_lo = sk_partial_segments(U, Gp, c_lo, kb_total) == 2 ? 1 : 2;
                    const int w_hi = (nseg > 1 && sk_partial_segments(U, Gp, c_hi, kb_total) == 2) ? 1 : 2;
                    fx_par[p][f][0] = tile; fx_par[p][f][1] = c_lo; fx_par[p][f][2] = nseg;
                    fx_par[p][f][3] = (cta == c_lo) ? 0 : w_lo + 2 * (cta - c_lo - 1);
                    fx_par[p][f][4] = (cta == c_lo) ? w_lo : (cta == c_hi ? w_hi : 2);
                    fx_par[p][f][5] = (nseg == 1) ? w_lo : w_lo + w_hi + 2 * (nseg - 2);
                }
            }
            fx_n[p] = n_fix;
        }
        __threadfence_block();
        fx_ready = 1;
    }
    if (sf.on && cta == 0 && warp >= 6 && warp < 14) {
        __shared__ float sel_dsh[SEL_SMALL_W];
        __shared__ int sel_flags[SEL_SMALL_W];
        __syncwarp();
        pdl_wait();
        step_select_inline(sf.sd, sf.a, (int)threadIdx.x - THREADS, 256, 2, sel_dsh, sel_flags);
    }

    // running counters of the roles (they continue across the projections of the chain)
    int p_units = 0;          // units the producer has requested / the MMA warp has consumed so far
    int seg = 0;              // accumulator segments so far (MMA warp and epilogue warps count the same sequence)
    unsigned bar_k = 0;       // grid-wide barriers so far (the same in every thread)
    const uint64_t pol = l2_policy_evict_first();

    // producer: weights of the first ring slots of projection p (nothing they depend on)
    auto producer_weights_ahead = [&](int p) {
        int kb_total; long long U, u_begin, u_end;
        range(p, kb_total, U, u_begin, u_end);
        const int n_units = (int)(u_end - u_begin);
        const int pre = min(stages, n_units);
        int tile = (int)(u_begin / kb_total), kb = (int)(u_begin - (long long)tile * kb_total);
        for (int i = 0; i < pre; ++i) {
            const int it = p_units + i;
            const int s = it % stages;
            if (it >= stages && !mbar_wait(empty0 + 8 * s, ((uint32_t)(it / stages) & 1u) ^ 1u, abort_flag)) return;
            mbar_expect_tx(full0 + 8 * s, STAGE_BYTES);
            tma_load_2d_hint(smem_base + s * STAGE_BYTES + A_BYTES, &maps.w[p], full0 + 8 * s, 0, (tile * kb_total + kb) * BLOCK_F, pol);
            if (++kb == kb_total) { kb = 0; ++tile; }
        }
    };

    if (warp == 0 && lane == 0) producer_weights_ahead(0);

    for (int p = 0; p < ca.n; ++p) {
        const ChainProb& P = ca.p[p];
        int kb_total; long long U, u_begin, u_end;
        range(p, kb_total, U, u_begin, u_end);
        const int n_units = (int)(u_end - u_begin);

        if (warp == 0) {
            if (lane == 0) {
                // ---- producer: activations of the slots whose weights are already on their way, then the rest
                bool ok = true;
                if (p == 0) pdl_wait();
                else {
                    ok = grid_counter_wait(ca.bar_counter, ca.bar_base + bar_k * (unsigned)G, abort_flag);
                    fence_async_global();      // rows written by other CTAs' ordinary stores, read by TMA from here on
                }
                const int pre = min(stages, n_units);
                int tile = (int)(u_begin / kb_total), kb = (int)(u_begin - (long long)tile * kb_total);
                for (int i = 0; i < pre && ok; ++i) {
                    const int s = (p_units + i) % stages;
                    tma_load_2d(smem_base + s * STAGE_BYTES, &maps.a[p], full0 + 8 * s, kb * BLOCK_K, 0);
                    if (++kb == kb_total) { kb = 0; ++tile; }
                }
                for (int i = pre; i < n_units && ok; ++i) {
                    const int it = p_units + i;
                    const int s = it % stages;
                    if (it >= stages && !mbar_wait(empty0 + 8 * s, ((uint32_t)(it / stages) & 1u) ^ 1u, abort_flag)) break;
                    const uint32_t dst = smem_base + s * STAGE_BYTES;
                    mbar_expect_tx(full0 + 8 * s, STAGE_BYTES);
                    tma_load_2d_hint(dst + A_BYTES, &maps.w[p], full0 + 8 * s, 0, (tile * kb_total + kb) * BLOCK_F, pol);
                    tma_load_2d(dst, &maps.a[p], full0 + 8 * s, kb * BLOCK_K, 0);
                    if (++kb == kb_total) { kb = 0; ++tile; }
                }
                p_units += n_units;
                if (p + 1 < ca.n) producer_weights_ahead(p + 1);      // while this projection drains and reduces
            }
        } else if (warp == 1) {
            if (lane == 0) {
                const uint32_t idesc = instr_desc_bf16(BLOCK_T, BLOCK_F);
                bool seg_start = true;
                int kb = (int)(u_begin % kb_total);
                for (int i = 0; i < n_units; ++i, kb = (kb + 1 == kb_total) ? 0 : kb + 1) {
                    const int it = p_units + i;
                    const int s = it % stages;
                    const uint32_t ph = (uint32_t)(it / stages) & 1u;
                    if (seg_start && seg > 1) {
                        if (!mbar_wait(accum_empty + 8 * (seg & 1), (uint32_t)((seg >> 1) - 1) & 1u, abort_flag)) break;
                        tc_fence_after();
                    }
                    if (!mbar_wait(full0 + 8 * s, ph, abort_flag)) break;
                    tc_fence_after();
                    const uint32_t sa = smem_base + s * STAGE_BYTES;
                    const uint64_t da = smem_desc_sw128(sa), dw = smem_desc_sw128(sa + A_BYTES);
#pragma unroll
                    for (int k = 0; k < BLOCK_K / UMMA_K; ++k)
                        umma_bf16(tmem_base + (uint32_t)((seg & 1) * BLOCK_F), da + (uint64_t)(k * 2), dw + (uint64_t)(k * 2), idesc,
                                  (!seg_start || k > 0) ? 1u : 0u);
                    umma_commit(empty0 + 8 * s);
                    seg_start = false;
                    if (kb == kb_total - 1 || i == n_units - 1) {
                        umma_commit(accum_full + 8 * (seg & 1));
                        ++seg;
                        seg_start = true;
                    }
                }
                p_units += n_units;
            }
        } else if (warp < 6) {
            // ---- epilogue warps: TMEM lane = token, column = feature
            if (p == 0) pdl_wait();
            trace_stamp(100 + P.epi, 64);
            const int q = warp & 3;
            const int t_local = q * 32 + lane;
            const uint32_t taddr0 = tmem_base + ((uint32_t)(q * 32) << 16);
            int Mv = -1;         // read once the first accumulator is ready: by then the producer has passed the grid
            bool live = false, warp_live = false;       // barrier, so a row count written earlier in this kernel is final
            long long u = u_begin;
            while (u < u_end) {
                const int tile = (int)(u / kb_total);
                const int k0 = (int)(u - (long long)tile * kb_total);
                const long long tile_end = (long long)(tile + 1) * kb_total;
                const long long seg_end = tile_end < u_end ? tile_end : u_end;
                const int k1 = (int)(seg_end - (long long)tile * kb_total);
                const int n0 = tile * BLOCK_F;
                const bool whole = (k0 == 0 && k1 == kb_total);
                if (!mbar_wait(accum_full + 8 * (seg & 1), (uint32_t)(seg >> 1) & 1u, abort_flag)) break;
                tc_fence_after();
                if (Mv < 0) {
                    Mv = P.e.m_count ? min(P.M, __ldcg(P.e.m_count)) : P.M;
                    live = t_local < Mv;
                    warp_live = q * 32 < Mv;
                }
                const uint32_t taddr = taddr0 + (uint32_t)((seg & 1) * BLOCK_F);
                if (P.e.accumulate) {
                    // this segment's part of the product goes straight onto the residual rows (whole or partial alike)
                    bool row_ok = live;
                    float* dst = P.e.out_f32 + (size_t)t_local * P.e.ld_out + n0;
                    if (live && P.epi == EPI_DOWN) {
                        // compacted row -> forward row; a selected window row of a refresh step lands in its packet row
                        // (which the RMSNorm staging before the gate/up projection has set to the residual row)
                        const int r0 = P.e.list ? __ldcg(P.e.list + t_local) : t_local;
                        const int4 rw = __ldg(reinterpret_cast<const int4*>(P.e.rows) + r0);       // {seq, pos, widx, aidx}
                        row_ok = rw.y >= 0;
                        dst = (P.e.within && rw.z >= 0) ? P.e.packet + ((size_t)rw.x * P.e.W_max + rw.z) * P.e.ld_out + n0
                                                        : P.e.out_f32 + (size_t)r0 * P.e.ld_out + n0;
                    }
                    if (warp_live) {
                        for (int c0 = 0; c0 < BLOCK_F; c0 += 64) {
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
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(accum_empty + 8 * (seg & 1));
                } else if (whole) {
                    if (warp_live) {
                        for (int c0 = 0; c0 < BLOCK_F; c0 += 16) {
                            float v[16];
                            tmem_ld16(taddr + (uint32_t)c0, v);
                            if (live) epi16_dyn<T>(P.epi, P.e, t_local, n0 + c0, v);
                        }
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(accum_empty + 8 * (seg & 1));
                } else {
                    const int which = (k0 == 0) ? 1 : 0;
                    float* part = ca.partial + ((size_t)(2 * cta + which) * BLOCK_T + t_local) * BLOCK_F;
                    if (warp_live) {
                        for (int c0 = 0; c0 < BLOCK_F; c0 += 64) {
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
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(accum_empty + 8 * (seg & 1));
                    __threadfence();
                    asm volatile("bar.sync 1, 128;" ::: "memory");
                    if (threadIdx.x == 64) atomicAdd(&ca.tile_counter[tile], 1);
                }
                ++seg;
                u = seg_end;
            }
        }
        // the MMA warp's other lanes and the producer's keep the counters in step
        if (warp == 0) p_units = __shfl_sync(0xffffffffu, p_units, 0);
        if (warp == 1) { p_units = __shfl_sync(0xffffffffu, p_units, 0); seg = __shfl_sync(0xffffffffu, seg, 0); }

        // ---- reduction of the split tiles of projection p (all warps)
        if (n_units > 0) {
            __syncwarp();
            if (p == 0) pdl_wait();
            const int Mv = P.e.m_count ? min(P.M, __ldcg(P.e.m_count)) : P.M;
            {
                const long long t0 = clock64();
                while (!fx_ready) { if (clock64() - t0 > WAIT_LIMIT_CYCLES) { *abort_flag = 1; break; } }
                __threadfence_block();
            }
            const int n_fix = fx_ready ? fx_n[p] : 0;
            if (n_fix > 0) {
                int fix_tile[2] = {0, 0}, f_lo[2] = {0, 0}, f_n[2] = {0, 0}, f_clo[2] = {0, 0}, f_nseg[2] = {1, 1};
#pragma unroll
                for (int f = 0; f < 2; ++f) {
                    if (f < n_fix) {
                        fix_tile[f] = fx_par[p][f][0]; f_clo[f] = fx_par[p][f][1]; f_nseg[f] = fx_par[p][f][2];
                        const int before = fx_par[p][f][3], mine = fx_par[p][f][4], w_all = fx_par[p][f][5];
                        const int n_items = max(0, min(BLOCK_T, Mv)) * (BLOCK_F / 16);
                        f_lo[f] = (n_items * before) / w_all;
                        f_n[f] = (n_items * (before + mine)) / w_all - f_lo[f];
                    }
                }
                const int total = f_n[0] + f_n[1];
                if ((int)threadIdx.x < total) {
                    const int f = (int)threadIdx.x < f_n[0] ? 0 : 1;
                    const int item = f_lo[f] + (int)threadIdx.x - (f ? f_n[0] : 0);
                    if (P.epi == EPI_RESID) epilogue_prefetch<T, EPI_RESID>(P.e, item / (BLOCK_F / 16), fix_tile[f] * BLOCK_F + (item % (BLOCK_F / 16)) * 16);
                    else if (P.epi == EPI_DOWN) epilogue_prefetch<T, EPI_DOWN>(P.e, item / (BLOCK_F / 16), fix_tile[f] * BLOCK_F + (item % (BLOCK_F / 16)) * 16);
                    else if (P.epi == EPI_SWIGLU) epilogue_prefetch<T, EPI_SWIGLU>(P.e, item / (BLOCK_F / 16), fix_tile[f] * BLOCK_F + (item % (BLOCK_F / 16)) * 16);
                    else epilogue_prefetch<T, EPI_QKV>(P.e, item / (BLOCK_F / 16), fix_tile[f] * BLOCK_F + (item % (BLOCK_F / 16)) * 16);
                }
                if (threadIdx.x == 64) {
                    const long long t0 = clock64();
                    int ok = 1;
                    for (int f = 0; f < n_fix && ok; ++f) {
                        while (ld_acquire_gpu(&ca.tile_counter[fix_tile[f]]) < f_nseg[f]) {
                            if (*abort_flag || clock64() - t0 > WAIT_LIMIT_CYCLES) { ok = 0; *abort_flag = 1; break; }
                            __nanosleep(64);
                        }
                    }
                    last_sh = ok;
                }
                __syncthreads();
                if ((P.epi == EPI_RESID || P.epi == EPI_DOWN) && last_sh && max(f_nseg[0], f_nseg[1]) > 4) {
                    for (int i4 = (int)threadIdx.x; i4 < 4 * total; i4 += FIX_THREADS) {
                        const int i = i4 >> 2;
                        const int f = i < f_n[0] ? 0 : 1;
                        const int item = f_lo[f] + i - (f ? f_n[0] : 0);
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
                                            ? __ldcg(reinterpret_cast<const float4*>(ca.partial + ((size_t)(2 * cc + wsl) * BLOCK_T + tl) * BLOCK_F + c0))
                                            : make_float4(0.f, 0.f, 0.f, 0.f);
                            }
#pragma unroll
                            for (int j = 0; j < 16; ++j) { acc.x += tv[j].x; acc.y += tv[j].y; acc.z += tv[j].z; acc.w += tv[j].w; }
                        }
                        epi4_dyn<T>(P.epi, P.e, tl, fix_tile[f] * BLOCK_F + c0, acc);
                    }
                } else if (last_sh) {
                    for (int i = (int)threadIdx.x; i < total; i += FIX_THREADS) {
                        const int f = i < f_n[0] ? 0 : 1;
                        const int item = f_lo[f] + i - (f ? f_n[0] : 0);
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
                                    const int wsl = (cc == c_lo) ? 1 : 0;
                                    const float4* ps = reinterpret_cast<const float4*>(
                                        ca.partial + ((size_t)(2 * cc + wsl) * BLOCK_T + tl) * BLOCK_F + c0);
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
                        epi16_dyn<T>(P.epi, P.e, tl, fix_tile[f] * BLOCK_F + c0, acc);
                    }
                }
                __syncthreads();
                if (threadIdx.x == 64 && last_sh) {
                    for (int f = 0; f < n_fix; ++f) {
                        const int tile = fix_tile[f];
                        const int prev = atomicAdd(&ca.tile_counter[ca.done_offset + tile], 1);
                        if (prev == f_nseg[f] - 1) { ca.tile_counter[tile] = 0; ca.tile_counter[ca.done_offset + tile] = 0; }
                    }
                }
            }
        }
        trace_stamp(200 + P.epi, 0);
        if (p + 1 == ca.n) break;

        // ---- every output row of projection p is stored: tell the grid; optional RMSNorm staging in between.
        // All barriers share one counter, so a CTA adds to it for barrier k + 1 only after barrier k has been passed
        // by the whole grid (otherwise early arrivals at k + 1 would be taken for late arrivals at k).
        auto arrive = [&]() {
            fence_async_global();
            __syncthreads();
            if (threadIdx.x == 0) {
                if (bar_k > 0) grid_counter_wait(ca.bar_counter, ca.bar_base + bar_k * (unsigned)G, abort_flag);
                __threadfence();
                grid_counter_arrive(ca.bar_counter, cta);
            }
            ++bar_k;
        };
        arrive();
        if (P.norm_after) {
            if (threadIdx.x == 0) post_ok = grid_counter_wait(ca.bar_counter, ca.bar_base + bar_k * (unsigned)G, abort_flag) ? 1 : 0;
            __syncthreads();
            if (post_ok) {
                for (int r = cta; r < P.post.n_rows; r += G) {
                    if (P.norm_after == 1)
                        prep_rows_row<T>(r, P.post.x, P.post.list, P.post.m_count, P.post.gain, P.post.eps, P.post.d, (T*)P.post.a_out, post_red,
                                         P.post.rows, const_cast<float*>(P.post.packet), P.post.sd.W_max);
                    else
                        prep_qkv_row<T>(P.post.sd, r, P.post.rows, P.post.x, P.post.hc, P.post.packet, P.post.patch, P.post.gain,
                                        P.post.eps, P.post.d, (T*)P.post.a_out, P.post.kvflag, post_red, P.post.ct);
                }
            }
            arrive();
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, ncols);
    if (threadIdx.x == 0 && abort_sh) atomicExch(ca.status, 1);
}

}  // namespace tc
}  // namespace ps
