// Skinny-M bf16 GEMM on 5th-generation tensor cores (tcgen05 + TMEM, operands staged by TMA).
//
//   out[m][n] = sum_k A[m][k] * W[n][k]      A: activations [M, K], W: weights [N_out, K]
//
// The decoding step multiplies a few dozen to a few hundred rows by every weight matrix, so
// the kernel is bound by streaming W from HBM.  The operands are therefore swapped: the
// weight tile (128 output features x 64 k) is the 128-row "A" operand of the MMA and the
// activation tile (NT tokens x 64 k, NT = 16..256) is the "B" operand.  The accumulator in
// tensor memory holds D^T: lane = output feature, column = token.  A small activation tile
// keeps shared memory for a deep pipeline of weight tiles, and no MMA rows are wasted on
// padding when only 32 rows are live.
//
// grid = (N_out / 128, ceil(M / NT), splits).  With splits > 1 every CTA writes its fp32
// partial tile to a workspace and the last CTA to arrive (per output tile) adds the partials in
// split order and runs the epilogue, which keeps results deterministic.
//
// Warp roles (192 threads): warp 0 = TMA producer, warp 1 = MMA issuer and TMEM owner,
// warps 2..5 = epilogue (one TMEM lane quarter each).  Every mbarrier wait is bounded; on
// time-out the CTA raises a status word, stops issuing work and leaves in an orderly way.
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace ps {
namespace tc {

constexpr int BLOCK_F = 128;   // output features per CTA (UMMA M)
constexpr int BLOCK_K = 64;    // bf16 elements per k block = one 128-byte swizzle row
constexpr int UMMA_K = 16;
constexpr int THREADS = 192;
constexpr long long WAIT_LIMIT_CYCLES = 4000000000LL;   // ~2 s

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
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
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128, N = n.
__host__ __device__ inline uint32_t instr_desc_bf16(int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(BLOCK_F >> 4) << 24);
}

struct GemmArgs {
    int M;          // rows of A that may be live (host bound)
    int N_out, K;
    int NT;         // tokens per tile: 16, 32, 64, 128 or 256
    int stages;
    int splits;
    float* partial;     // [splits][tiles_f][tiles_t][NT][128] fp32 (splits > 1)
    int* tile_counter;  // [tiles_f * tiles_t], zero before launch, zero again after
    int* status;        // set to 1 on a wait time-out
};

template <typename T, int EPI>
__global__ void __launch_bounds__(THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_a,
               GemmArgs g, EpiArgs e) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bars[2 * 12 + 1];
    __shared__ uint32_t tmem_base_sh;
    __shared__ int abort_sh;
    __shared__ int last_sh;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tile_f = blockIdx.x, tile_t = blockIdx.y, split = blockIdx.z;
    const int t0 = tile_t * g.NT;
    const int Mv = e.m_count ? min(g.M, *e.m_count) : g.M;
    if (t0 >= Mv) return;     // whole tile beyond the live rows (uniform over the CTA)

    const int kb_total = g.K / BLOCK_K;
    const int kb_begin = (int)(((long long)kb_total * split) / g.splits);
    const int kb_end = (int)(((long long)kb_total * (split + 1)) / g.splits);
    const int n_kb = kb_end - kb_begin;

    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t w_bytes = BLOCK_F * BLOCK_K * 2, a_bytes = (uint32_t)g.NT * BLOCK_K * 2;
    const uint32_t stage_bytes = w_bytes + a_bytes;
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t full0 = smem_u32(&bars[0]), empty0 = smem_u32(&bars[12]), accum_bar = smem_u32(&bars[24]);
    const uint32_t ncols = g.NT < 32 ? 32u : (uint32_t)g.NT;

    if (threadIdx.x == 0) {
        for (int s = 0; s < g.stages; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
        mbar_init(accum_bar, 1);
        abort_sh = 0;
        last_sh = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32(&tmem_base_sh), ncols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_sh;
    volatile int* abort_flag = &abort_sh;

    if (warp == 0) {
        if (lane == 0) {
            for (int i = 0; i < n_kb; ++i) {
                const int s = i % g.stages;
                const uint32_t ph = (uint32_t)(i / g.stages) & 1u;
                if (!mbar_wait(empty0 + 8 * s, ph ^ 1u, abort_flag)) break;
                const uint32_t dst = smem_base + s * stage_bytes;
                mbar_expect_tx(full0 + 8 * s, stage_bytes);
                tma_load_2d(dst, &map_w, full0 + 8 * s, (kb_begin + i) * BLOCK_K, tile_f * BLOCK_F);
                tma_load_2d(dst + w_bytes, &map_a, full0 + 8 * s, (kb_begin + i) * BLOCK_K, t0);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = instr_desc_bf16(g.NT);
            bool ok = true;
            for (int i = 0; i < n_kb && ok; ++i) {
                const int s = i % g.stages;
                const uint32_t ph = (uint32_t)(i / g.stages) & 1u;
                ok = mbar_wait(full0 + 8 * s, ph, abort_flag);
                if (!ok) break;
                tc_fence_after();
                const uint32_t wa = smem_base + s * stage_bytes;
                const uint64_t dw = smem_desc_sw128(wa), da = smem_desc_sw128(wa + w_bytes);
#pragma unroll
                for (int k = 0; k < BLOCK_K / UMMA_K; ++k)
                    umma_bf16(tmem_base, dw + (uint64_t)(k * 2), da + (uint64_t)(k * 2), idesc, (i > 0 || k > 0) ? 1u : 0u);
                umma_commit(empty0 + 8 * s);
            }
            umma_commit(accum_bar);     // arrives once every MMA issued so far has finished
        }
    } else {
        // ---- epilogue warps: quarter q of the TMEM lanes = features 32q .. 32q+31 of the tile
        const int q = warp & 3;
        const int f_local = q * 32 + lane;
        const int n = tile_f * BLOCK_F + f_local;
        const bool got = mbar_wait(accum_bar, 0, abort_flag);
        tc_fence_after();
        if (got) {
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16);
            const int nt_live = min(g.NT, Mv - t0);
            if (g.splits == 1) {
                for (int c0 = 0; c0 < nt_live; c0 += 16) {
                    float v[16];
                    tmem_ld16(taddr + (uint32_t)c0, v);
#pragma unroll
                    for (int c = 0; c < 16; ++c) {
                        const float partner = __shfl_xor_sync(0xffffffffu, v[c], 1);
                        const int m = t0 + c0 + c;
                        if (!(lane & 1) && m < Mv && n < g.N_out) epilogue_pair<T, EPI>(e, m, n, v[c], partner);
                    }
                }
            } else {
                float* part = g.partial + ((((size_t)split * gridDim.x + tile_f) * gridDim.y + tile_t) * g.NT) * BLOCK_F;
                for (int c0 = 0; c0 < nt_live; c0 += 16) {
                    float v[16];
                    tmem_ld16(taddr + (uint32_t)c0, v);
#pragma unroll
                    for (int c = 0; c < 16; ++c) part[(size_t)(c0 + c) * BLOCK_F + f_local] = v[c];
                }
                __threadfence();
            }
        }
    }

    if (g.splits > 1) {
        // last CTA of this output tile sums the partials (fixed order) and runs the epilogue
        __syncthreads();
        if (threadIdx.x == 0) {
            const int prev = atomicAdd(&g.tile_counter[tile_f * gridDim.y + tile_t], 1);
            last_sh = (prev == g.splits - 1);
        }
        __syncthreads();
        if (last_sh && warp >= 2 && !abort_sh) {
            __threadfence();
            const int q = warp & 3;
            const int f_local = q * 32 + lane;
            const int n = tile_f * BLOCK_F + f_local;
            const int nt_live = min(g.NT, Mv - t0);
            for (int c = 0; c < nt_live; ++c) {
                float acc = 0.f;
                for (int sp = 0; sp < g.splits; ++sp) {
                    const float* part = g.partial + ((((size_t)sp * gridDim.x + tile_f) * gridDim.y + tile_t) * g.NT) * BLOCK_F;
                    acc += __ldcg(part + (size_t)c * BLOCK_F + f_local);
                }
                const float partner = __shfl_xor_sync(0xffffffffu, acc, 1);
                const int m = t0 + c;
                if (!(lane & 1) && n < g.N_out) epilogue_pair<T, EPI>(e, m, n, acc, partner);
            }
        }
        if (last_sh && threadIdx.x == 0) g.tile_counter[tile_f * gridDim.y + tile_t] = 0;
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, ncols);
    if (threadIdx.x == 0 && abort_sh) atomicExch(g.status, 1);
}

}  // namespace tc
}  // namespace ps
