// Bidirectional attention rows with drift on 5th-generation tensor cores (Eq. 3, Eq. 4): bf16 models,
// head_dim 128, up to 2048 keys.  One pass over K.
//
// Work item of a CTA: 128 query rows x 1 head x a range of 128 or 256 keys.  The key ranges of one
// (row tile, head) form a thread-block cluster (1..8 CTAs), so that a single block of 32 active rows still
// pulls K/V through 4 x n_heads SMs.
//
//   S = Q K^T      tcgen05.mma 128 x 128 x 16, Q and K tiles brought by TMA (128-byte swizzle), S in tensor memory
//   statistics     eight warps read S from tensor memory (lane = row): the range's maximum and sum, which every
//                  CTA PUSHES into its peers' shared memory (st.shared::cluster + a remote mbarrier arrival), so
//                  each CTA gets the row's log-sum-exp without a cluster-wide barrier; then p = 2^(t - lse)
//                  (normalised BEFORE it is rounded to bf16, the rounding point of a plain implementation),
//                  A = sum p (s - s_old) against the stored row, the new stored row s, and P written back to
//                  shared memory in the operand layout
//   O = P V        tcgen05.mma with V as an MN-major operand (keys x head_dim as it lies in the cache)
//   combine        every CTA owns a share of the rows; the others push their partial outputs and drift sums of
//                  those rows into the owner's shared memory; the owner adds them in rank order and stores
//
// Stored rows.  A recorded row is kept as its scaled scores s_j = q.k_j / sqrt(d) (natural-log units) plus
// one log-sum-exp per row; the log-probability is s_j - lse.  KL, the new stored row and P V then need no
// second pass over K:
//     KL(p || p_old) = sum_j p_j (s_j - s_old_j) - (lse - lse_old)
// Both terms are exactly zero when nothing changed (same bits in, same bits out), so unchanged rows have
// zero drift.  Every mbarrier is used once (one tile per CTA: no phases); all waits are bounded.
#pragma once
#include "gemm_tc.cuh"

namespace ps {
namespace atc {

using namespace tc;

constexpr int ROWS = 128;                 // query rows per CTA (UMMA M)
constexpr int KEYS = 128;                 // keys per S tile (UMMA N)
constexpr int DH = 128;
constexpr int MAX_KT = 2;                 // S tiles per CTA
constexpr int MAX_CL = 8;                 // CTAs per cluster (portable limit)
constexpr int MAX_N = KEYS * MAX_KT * MAX_CL;
constexpr int THREADS = 320;              // warp 0: TMA, warp 1: MMA + tensor memory, warps 2..9: statistics / epilogue
constexpr uint32_t BOX_BYTES = 128 * 64 * 2;     // one [128][64] bf16 box = 16 KB
constexpr uint32_t XCH_BYTES = 40 * 1024;        // receive area in front of the operand tiles (with the Q tile: 72 KB)
constexpr int OROW = DH + 4;                     // floats per exchanged row: 128 outputs, the two drift sums, padding
constexpr uint32_t STAGE_PAD = 4 * 1024;         // the staging area of the partial outputs overhangs K0 + V0 by 2 KB
constexpr float LOG2E_F = 1.4426950408889634f;
constexpr float LN2_F = 0.6931471805599453f;

__host__ __device__ constexpr size_t smem_bytes(int kt) { return XCH_BYTES + (size_t)(2 + 4 * kt) * BOX_BYTES + STAGE_PAD + 1024; }

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y, int z) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "r"(z)
        : "memory");
}
// MN-major operand tile with 128-byte swizzle: rows of 64 elements (128 bytes) indexed by k, 8-row groups 1024
// bytes apart, the next 64 elements along MN `lbo_bytes` further on
__device__ __forceinline__ uint64_t smem_desc_mn_sw128(uint32_t addr, uint32_t lbo_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)(lbo_bytes >> 4) << 16;
    d |= (uint64_t)(1024u >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float ld_dsmem_f(uint32_t addr) {
    float v;
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ void bar_sync_epi() { asm volatile("bar.sync 1, 256;" ::: "memory"); }
// ---- exchange inside the cluster: plain stores into a peer's shared memory, then an arrival on the peer's mbarrier
// with release semantics at cluster scope; the peer's wait acquires at cluster scope
__device__ __forceinline__ void st_dsmem_f2(uint32_t addr, float x, float y) {
    asm volatile("st.shared::cluster.v2.f32 [%0], {%1, %2};" ::"r"(addr), "f"(x), "f"(y) : "memory");
}
__device__ __forceinline__ void st_dsmem_u4(uint32_t addr, uint32_t x, uint32_t y, uint32_t z, uint32_t w) {
    asm volatile("st.shared::cluster.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(x), "r"(y), "r"(z), "r"(w) : "memory");
}
__device__ __forceinline__ void st_dsmem_f(uint32_t addr, float x) {
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(addr), "f"(x) : "memory");
}
__device__ __forceinline__ void mbar_arrive_remote(uint32_t remote_bar) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(remote_bar) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok;
}
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    if (mbar_try_wait_cluster(bar, parity)) return true;
    const long long t0 = clock64();
    while (true) {
        for (int i = 0; i < 64; ++i)
            if (mbar_try_wait_cluster(bar, parity)) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > WAIT_LIMIT_CYCLES) { *abort_flag = 1; return false; }
    }
}

// POLESTAR_TRACE_ATTN builds (on top of POLESTAR_TRACE; the probes' own global accesses perturb what they measure,
// so the ordinary trace build leaves them out): cycle counter of CTA (0, 0) at point k, for the producer (thread 0, slots 40+), the MMA thread
// (32, slots 50+), an epilogue thread of rows 64.. (64, slots 0+) and one of rows 0.. (128, slots 20+)
#if defined(POLESTAR_TRACE) && defined(POLESTAR_TRACE_ATTN)
__device__ __forceinline__ void dbg_clock(int k) {
    long long* t = g_trace_buf;
    if (!t || blockIdx.x != 0 || blockIdx.y != 0) return;
    const int th = threadIdx.x;
    const int base = th == 64 ? 0 : th == 128 ? 20 : th == 0 ? 40 : th == 32 ? 50 : -1;
    if (base >= 0) t[8100 + base + k] = clock64();
}
#else
__device__ __forceinline__ void dbg_clock(int) {}
#endif

struct Args {
    AttnArgs a;
    int rows_per_seq;       // forward rows per sequence (stand-alone: n_rows)
    int tiles_per_seq;      // 128-row tiles per sequence
    int kt;                 // S tiles (128 keys) per CTA: 1 or 2
    int cl;                 // CTAs per cluster = key ranges per (row tile, head)
    int* status;            // set to 1 when a bounded wait gave up (null: nowhere to report)
};

// bulk copy from this CTA's shared memory into a peer's; completion is counted in bytes on the PEER's mbarrier
__device__ __forceinline__ void bulk_copy_to_peer(uint32_t dst_cluster, uint32_t src_cta, uint32_t bytes, uint32_t bar_cluster) {
    asm volatile("cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst_cluster), "r"(src_cta), "r"(bytes), "r"(bar_cluster) : "memory");
}

__global__ void __launch_bounds__(THREADS, 1)
attention_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                    const __grid_constant__ CUtensorMap map_v, Args g) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bars[6 + 3 * MAX_KT];      // q, s, o, x (statistics in), y (partial rows in), spare, then k[j], v[j], p[j]
    __shared__ uint32_t tmem_base_sh;
    __shared__ int abort_sh;
    __shared__ float* prev_sh[ROWS];
    __shared__ float* lsep_sh[ROWS];
    __shared__ int valid_sh[ROWS];
    __shared__ float2 half_ml[2][ROWS];            // (maximum, sum) of each column half
    __shared__ float2 xch_ml[MAX_CL][ROWS];        // received: key range c's (maximum m, sum of 2^(t - m)) of every row
    __shared__ float dlse_sh[ROWS];                // owned rows: lse - lse_old (natural-log units)

    const AttnArgs& a = g.a;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int cl = g.cl, kt = g.kt;
    const int rank = (int)cluster_rank();
    const int bx = blockIdx.x / cl;
    const int seq = bx / g.tiles_per_seq, tile = bx - seq * g.tiles_per_seq;
    const int h = blockIdx.y;
    const int g_kv = (h * a.n_kv) / a.n_heads;
    const int dq = a.n_heads * DH;
    const int row0 = seq * g.rows_per_seq + tile * ROWS;
    const int n_in_tile = min(ROWS, g.rows_per_seq - tile * ROWS);
    const int kv_seq = a.rows ? seq : 0;
    const int key0 = rank * kt * KEYS;
    const int n_kt = min(kt, (a.N - key0 + KEYS - 1) / KEYS);      // S tiles of this CTA that hold any key (>= 1)
    const int rb = (ROWS + cl - 1) / cl;                            // rows finished ("owned") by each CTA of the cluster
    const int my_rows = max(0, min(ROWS, (rank + 1) * rb) - rank * rb);

    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t smem_base = smem_u32(smem);
    // receive area for the peers' partial rows [cl][rb][OROW] fp32: the first XCH_BYTES plus the Q tile, which is free
    // by the time any peer can have an output (a peer needs this CTA's statistics first, and those follow its S)
    const uint32_t ox_s = smem_base;
    const uint32_t q_s = smem_base + XCH_BYTES;                      // 2 boxes
    auto k_s = [&](int j) { return q_s + (uint32_t)(2 + 4 * j) * BOX_BYTES; };        // 2 boxes, later P_j
    auto v_s = [&](int j) { return q_s + (uint32_t)(4 + 4 * j) * BOX_BYTES; };        // 2 boxes
    // staging of this CTA's partial rows [128][OROW] once the operand tiles are spent: from K0 on
    const uint32_t st_s = k_s(0);
    float* const st_p = reinterpret_cast<float*>(smem + XCH_BYTES + 2 * BOX_BYTES);
    const uint32_t bar_q = smem_u32(&bars[0]), bar_s = smem_u32(&bars[1]), bar_o = smem_u32(&bars[2]);
    const uint32_t bar_x = smem_u32(&bars[3]), bar_y = smem_u32(&bars[4]);
    auto bar_k = [&](int j) { return smem_u32(&bars[6 + 3 * j]); };
    auto bar_v = [&](int j) { return smem_u32(&bars[7 + 3 * j]); };
    auto bar_p = [&](int j) { return smem_u32(&bars[8 + 3 * j]); };
    const uint32_t ncols = kt == 1 ? 256u : 512u;
    const uint32_t o_col = (uint32_t)(kt * KEYS);

    if (threadIdx.x == 0) {
        mbar_init(bar_q, 1); mbar_init(bar_s, 1); mbar_init(bar_o, 1);
        mbar_init(bar_x, (uint32_t)(cl * ROWS));             // every row of every key range
        mbar_init(bar_y, 1);                                 // armed below with the bytes the peers will copy in
        for (int j = 0; j < MAX_KT; ++j) { mbar_init(bar_k(j), 1); mbar_init(bar_v(j), 1); mbar_init(bar_p(j), 8); }
        abort_sh = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        mbar_expect_tx(bar_y, (uint32_t)(cl * my_rows * OROW * 4));
    }
    if (warp == 1) tmem_alloc(smem_u32(&tmem_base_sh), ncols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    pdl_trigger();
    dbg_clock(0);
    // peers arrive on this CTA's barriers and write its shared memory: announce that both exist (the matching wait
    // comes right before the first remote access, by which time it costs nothing)
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    const uint32_t tmem_base = tmem_base_sh;
    volatile int* abort_flag = &abort_sh;

    if (warp == 0) {
        if (lane == 0) {
            // Key tiles outside [dirty_lo, dirty_hi) were last written by an earlier forward, which the host has
            // waited for: their K / V can be on their way while the previous kernel still runs.
            auto tile_clean = [&](int j) {
                const int lo = key0 + j * KEYS, hi = lo + KEYS;
                return hi <= a.dirty_lo || lo >= a.dirty_hi;
            };
            auto load_k = [&](int j) {
                mbar_expect_tx(bar_k(j), 2 * BOX_BYTES);
                for (int kb = 0; kb < 2; ++kb)
                    tma_load_3d(k_s(j) + kb * BOX_BYTES, &map_k, bar_k(j), g_kv * DH + kb * 64, key0 + j * KEYS, kv_seq);
            };
            auto load_v = [&](int j) {
                mbar_expect_tx(bar_v(j), 2 * BOX_BYTES);
                for (int kb = 0; kb < 2; ++kb)
                    tma_load_3d(v_s(j) + kb * BOX_BYTES, &map_v, bar_v(j), g_kv * DH + kb * 64, key0 + j * KEYS, kv_seq);
            };
            for (int j = 0; j < n_kt; ++j) if (tile_clean(j)) load_k(j);
            for (int j = 0; j < n_kt; ++j) if (tile_clean(j)) load_v(j);
            // q, and the K/V rows written this step, come from the projection that ran just before
            pdl_wait();
            trace_stamp(7);
            dbg_clock(1);
            mbar_expect_tx(bar_q, 2 * BOX_BYTES);
            for (int kb = 0; kb < 2; ++kb) tma_load_2d(q_s + kb * BOX_BYTES, &map_q, bar_q, h * DH + kb * 64, row0);
            for (int j = 0; j < n_kt; ++j) if (!tile_clean(j)) load_k(j);
            for (int j = 0; j < n_kt; ++j) if (!tile_clean(j)) load_v(j);
        }
        __syncwarp();
        asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc_s = instr_desc_bf16(ROWS, KEYS);
            const uint32_t idesc_o = instr_desc_bf16(ROWS, DH) | (1u << 16);       // B (= V) is MN-major
            bool ok = mbar_wait(bar_q, 0, abort_flag);
            dbg_clock(1);
            for (int j = 0; j < n_kt && ok; ++j) {
                ok = mbar_wait(bar_k(j), 0, abort_flag);
                if (!ok) break;
                tc_fence_after();
                dbg_clock(2);
#pragma unroll
                for (int k = 0; k < DH / UMMA_K; ++k) {
                    const uint64_t da = smem_desc_sw128(q_s + (k >> 2) * BOX_BYTES) + (uint64_t)((k & 3) * 2);
                    const uint64_t db = smem_desc_sw128(k_s(j) + (k >> 2) * BOX_BYTES) + (uint64_t)((k & 3) * 2);
                    umma_bf16(tmem_base + (uint32_t)(j * KEYS), da, db, idesc_s, k > 0 ? 1u : 0u);
                }
            }
            umma_commit(bar_s);          // (also on failure: the statistics warps then see the abort flag)
            dbg_clock(3);
            for (int j = 0; j < n_kt && ok; ++j) {
                ok = mbar_wait(bar_v(j), 0, abort_flag) && mbar_wait(bar_p(j), 0, abort_flag);
                if (!ok) break;
                tc_fence_after();
                dbg_clock(4);
#pragma unroll
                for (int k = 0; k < KEYS / UMMA_K; ++k) {
                    // A = P_j: K-major, 64 keys per 128-byte row;  B = V_j: 16 keys = two 8-row groups further down
                    const uint64_t da = smem_desc_sw128(k_s(j) + (k >> 2) * BOX_BYTES) + (uint64_t)((k & 3) * 2);
                    const uint64_t db = smem_desc_mn_sw128(v_s(j) + (uint32_t)k * 2048u, BOX_BYTES);
                    umma_bf16(tmem_base + o_col, da, db, idesc_o, (j > 0 || k > 0) ? 1u : 0u);
                }
            }
            umma_commit(bar_o);
            dbg_clock(5);
        }
        __syncwarp();
        asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    } else {
        // ---- statistics / epilogue warps: TMEM lane = row; the two warps of a lane quarter split the columns ----
        const int ew = warp - 2;
        const int quarter = warp & 3;
        const int half = ew >> 2;
        const int row = quarter * 32 + lane;
        const int owner = row / rb, lrow = row - owner * rb;
        const uint32_t taddr0 = tmem_base + ((uint32_t)(quarter * 32) << 16);
        pdl_wait();            // the row table, q and the stored rows all come from earlier kernels of the stream
        dbg_clock(1);
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
        // tensor-memory loads are warp-wide (.sync.aligned): whether a warp reads at all is decided per warp, and
        // only what a lane does with its row depends on that row
        const bool warp_valid = __any_sync(0xffffffffu, valid) != 0;
        const bool use_old = prev != nullptr && a.record_kl != 0;
        const bool vec = (a.N & 3) == 0;
        // the stored row of the first key tile and (owner only) the stored log-sum-exp are read now, long before
        // they are needed: their latency hides behind the wait for S
        float old[64];
#pragma unroll
        for (int i = 0; i < 64; ++i) old[i] = 0.f;
        auto load_old = [&](int j) {
            const int kb = key0 + j * KEYS + half * 64;
            if (vec) {
#pragma unroll
                for (int i = 0; i < 64; i += 4)
                    if (kb + i < a.N) {
                        const float4 o4 = __ldcg(reinterpret_cast<const float4*>(prev + kb + i));
                        old[i] = o4.x; old[i + 1] = o4.y; old[i + 2] = o4.z; old[i + 3] = o4.w;
                    }
            } else {
#pragma unroll
                for (int i = 0; i < 64; ++i)
                    if (kb + i < a.N) old[i] = __ldcg(prev + kb + i);
            }
        };
        if (use_old) load_old(0);
        float lse_old = 0.f;
        const bool owns = half == 0 && owner == rank;
        if (owns && lsep_sh[row] && a.record_kl) lse_old = __ldcg(lsep_sh[row]);
        const float scale2 = a.scale * LOG2E_F;
        dbg_clock(2);
        bool ok = mbar_wait(bar_s, 0, abort_flag) && !*abort_flag;
        ok = __all_sync(0xffffffffu, ok) != 0;
        tc_fence_after();
        dbg_clock(3);
        // pass A: (maximum, sum) of this thread's columns with a running maximum, then of the CTA's key range
        float mx = -INFINITY, l = 0.f;
        if (ok && warp_valid) {
            for (int j = 0; j < n_kt; ++j) {
                uint32_t r[4][16];
#pragma unroll
                for (int u = 0; u < 4; ++u) tmem_ld16_issue(taddr0 + (uint32_t)(j * KEYS + half * 64 + 16 * u), r[u]);
                tmem_ld_wait();
                const int kb = key0 + j * KEYS + half * 64;
                float tm = -INFINITY;
#pragma unroll
                for (int u = 0; u < 4; ++u)
#pragma unroll
                    for (int i = 0; i < 16; ++i)
                        if (kb + 16 * u + i < a.N) tm = fmaxf(tm, __uint_as_float(r[u][i]));
                tm *= scale2;      // scale2 > 0: the maximum commutes with it
                const float nm = fmaxf(mx, tm);
                float sum = 0.f;
                if (nm > -INFINITY) {
#pragma unroll
                    for (int u = 0; u < 4; ++u)
#pragma unroll
                        for (int i = 0; i < 16; ++i)
                            if (kb + 16 * u + i < a.N) sum += ex2(__uint_as_float(r[u][i]) * scale2 - nm);
                    l = l * ex2(mx - nm) + sum;       // (mx = -inf: l is 0 and 2^(-inf) = 0)
                }
                mx = nm;
            }
        }
        dbg_clock(4);
        half_ml[half][row] = make_float2(mx, l);
        bar_sync_epi();
        __syncwarp();
        asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");      // every peer's barriers and memory exist
        dbg_clock(5);
        if (half == 0) {
            const float2 h0 = half_ml[0][row], h1 = half_ml[1][row];
            const float m = fmaxf(h0.x, h1.x);
            float sum = 0.f;
            if (h0.y > 0.f) sum += h0.y * ex2(h0.x - m);
            if (h1.y > 0.f) sum += h1.y * ex2(h1.x - m);
            // this key range's (maximum, sum) of the row goes to every CTA of the cluster, this one included
            const uint32_t slot = smem_u32(&xch_ml[rank][row]);
            for (int c = 0; c < cl; ++c) st_dsmem_f2(dsmem_addr(slot, (uint32_t)c), m, sum);
            for (int c = 0; c < cl; ++c) mbar_arrive_remote(dsmem_addr(bar_x, (uint32_t)c));
        }
        dbg_clock(6);
        ok = mbar_wait_cluster(bar_x, 0, abort_flag) && ok;
        ok = __all_sync(0xffffffffu, ok) != 0;
        dbg_clock(7);
        // the row's log-sum-exp from all key ranges, in rank order (every CTA gets the same bits)
        float lse2;
        {
            float M = -INFINITY;
            for (int c = 0; c < cl; ++c) M = fmaxf(M, xch_ml[c][row].x);
            float L = 0.f;
            for (int c = 0; c < cl; ++c) {
                const float2 ml = xch_ml[c][row];
                if (ml.y > 0.f) L = fmaf(ml.y, ex2(ml.x - M), L);
            }
            lse2 = M + log2f(L);
        }
        if (owns) {
            // the owner of a row keeps its log-sum-exp (natural-log units, like the stored rows)
            float* lsep = lsep_sh[row];
            const float lse = lse2 * LN2_F;
            dlse_sh[row] = lse - lse_old;
            if (lsep && valid) *lsep = lse;
        }
        dbg_clock(8);
        // pass B: probabilities (normalised before they are rounded to bf16), drift sum, the new stored row, P
        float A = 0.f;
        for (int j = 0; j < n_kt; ++j) {
            if (ok && warp_valid) {
                if (j > 0 && use_old) load_old(j);
                uint32_t r[4][16];
#pragma unroll
                for (int u = 0; u < 4; ++u) tmem_ld16_issue(taddr0 + (uint32_t)(j * KEYS + half * 64 + 16 * u), r[u]);
                tmem_ld_wait();
                const int kb = key0 + j * KEYS + half * 64;
                const uint32_t p_row = k_s(j) + (uint32_t)half * BOX_BYTES + (uint32_t)row * 128u;
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    float s_nat[16], pr[16];
                    const int k16 = kb + 16 * u;
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const bool in = valid && (k16 + i < a.N);
                        const float t = __fmul_rn(__uint_as_float(r[u][i]), scale2);     // (rounded products, never fused into the
                                                                                         // subtraction from the stored value below)
                        const float p = in ? ex2(t - lse2) : 0.f;      // rows that are not valid hand zeros to the tensor core
                        s_nat[i] = __fmul_rn(t, LN2_F);
                        if (use_old && in) A = fmaf(p, s_nat[i] - old[16 * u + i], A);
                        pr[i] = p;
                    }
                    if (prev && valid) {
                        if (vec) {
#pragma unroll
                            for (int i = 0; i < 16; i += 4)
                                if (k16 + i < a.N)
                                    __stcg(reinterpret_cast<float4*>(prev + k16 + i), make_float4(s_nat[i], s_nat[i + 1], s_nat[i + 2], s_nat[i + 3]));
                        } else {
#pragma unroll
                            for (int i = 0; i < 16; ++i)
                                if (k16 + i < a.N) __stcg(prev + k16 + i, s_nat[i]);
                        }
                    }
                    // P as the A operand of P V: row `row`, 16-byte chunks 2u and 2u + 1 of the 128-byte row, XOR-swizzled
#pragma unroll
                    for (int c = 0; c < 2; ++c) {
                        uint32_t w[4];
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            __nv_bfloat162 b = __floats2bfloat162_rn(pr[8 * c + 2 * i], pr[8 * c + 2 * i + 1]);
                            w[i] = *reinterpret_cast<uint32_t*>(&b);
                        }
                        const uint32_t dst = p_row + (uint32_t)(((2 * u + c) ^ (row & 7)) << 4);
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]) : "memory");
                    }
                }
            }
            // P_j is complete for this warp's rows (a warp without any valid row leaves what the K tile held there:
            // finite bf16 values whose output rows are never written)
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_p(j));
        }
        dbg_clock(9);
        // partial rows of this key range -> staging (16-byte chunk j of a row at chunk j ^ (local row & 31): neither
        // the writers nor the reader meet bank conflicts), then one bulk copy per owner
        ok = mbar_wait(bar_o, 0, abort_flag) && ok && !*abort_flag;
        ok = __all_sync(0xffffffffu, ok) != 0;
        tc_fence_after();
        dbg_clock(10);
        if (ok && warp_valid) {
            uint32_t r[4][16];
#pragma unroll
            for (int u = 0; u < 4; ++u) tmem_ld16_issue(taddr0 + o_col + (uint32_t)(half * 64 + 16 * u), r[u]);
            tmem_ld_wait();
            float* dst = st_p + (size_t)row * OROW;
#pragma unroll
            for (int u = 0; u < 4; ++u)
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int chunk = half * 16 + 4 * u + i;
                    *reinterpret_cast<uint4*>(dst + ((chunk ^ (lrow & 31)) << 2)) = make_uint4(r[u][4 * i], r[u][4 * i + 1], r[u][4 * i + 2], r[u][4 * i + 3]);
                }
        }
        st_p[(size_t)row * OROW + DH + half] = A;
        tc_fence_before();
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // the bulk copies read what was just written
        bar_sync_epi();
        dbg_clock(11);
        if (ew == 0 && lane == 0) {
            for (int c = 0; c < cl; ++c) {
                const int n_c = max(0, min(ROWS, (c + 1) * rb) - c * rb);
                bulk_copy_to_peer(dsmem_addr(ox_s + (uint32_t)(rank * rb * OROW * 4), (uint32_t)c), st_s + (uint32_t)(c * rb * OROW * 4),
                                  (uint32_t)(n_c * OROW * 4), dsmem_addr(bar_y, (uint32_t)c));
            }
        }
        // ---- the owned rows: add the key ranges' contributions in rank order, store ----------------------------
        ok = mbar_wait_cluster(bar_y, 0, abort_flag) && ok && !*abort_flag;
        ok = __all_sync(0xffffffffu, ok) != 0;
        dbg_clock(12);
        if (ok) {
            const float* ox = reinterpret_cast<const float*>(smem);
            for (int lr = ew; lr < my_rows; lr += 8) {
                const int orow = rank * rb + lr;
                if (!valid_sh[orow]) continue;
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
                float sa = 0.f;
                for (int c = 0; c < cl; ++c) {
                    const float* src = ox + (size_t)(c * rb + lr) * OROW;
                    const float4 v = *reinterpret_cast<const float4*>(src + ((lane ^ (lr & 31)) << 2));
                    acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
                    sa += src[DH] + src[DH + 1];
                }
                if (a.out) {
                    __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y), hi = __floats2bfloat162_rn(acc.z, acc.w);
                    uint2 u;
                    u.x = *reinterpret_cast<uint32_t*>(&lo); u.y = *reinterpret_cast<uint32_t*>(&hi);
                    *reinterpret_cast<uint2*>((__nv_bfloat16*)a.out + (size_t)(row0 + orow) * dq + h * DH + lane * 4) = u;
                }
                if (lane == 0 && a.kl)
                    a.kl[(size_t)(row0 + orow) * a.n_heads + h] = (lsep_sh[orow] && a.record_kl) ? sa - dlse_sh[orow] : 0.f;
            }
        }
        dbg_clock(13);
    }

    // The peers' copies out of this CTA's staging area are complete once every owner has all its bytes: the cluster
    // meets once more before anybody leaves.
    __syncwarp();
    cluster_sync_all();
    dbg_clock(14);
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, ncols);
    trace_stamp(311, 64);
    if (threadIdx.x == 0 && abort_sh && g.status) atomicExch(g.status, 1);
}

}  // namespace atc
}  // namespace ps
