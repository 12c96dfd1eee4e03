// Bidirectional attention rows with drift for bf16 models, head_dim 128 (Eq. 3, Eq. 4).
//
// Three kernels share the tile helpers below; launch_attention_mma picks one from the row and key counts:
//   attention_sp_kernel   16 query rows x 1 head per CTA, keys split over the warps, scores kept in registers
//                         (N <= 1024): K is read once.  With a single block of rows the keys of a (row tile, head)
//                         are further split over a cluster of two CTAs.
//   attention_mma_kernel  the same tiling for N > 1024 with few rows: two passes over K (below).
//   attention_big_kernel  64 query rows x 1 head per CTA for entry forwards, batches and long sequences.
// The two-pass form: pass 1 gives every row's log-sum-exp (online max/sum per warp, combined across warps);
// pass 2 recomputes the scores, forms logp = s - lse, p = exp(logp), accumulates
// KL(p || stored row), overwrites the stored row with logp and accumulates p V.
// Two passes keep logp exact (no running rescale of the stored rows); the second read of K
// comes from L2.  Tensor-core path: warp-level mma.sync m16n8k16 (bf16 in, fp32 accumulate).
#pragma once
#include "kernels.cuh"

namespace ps {

constexpr int AT_BM = 16;        // query rows per CTA
constexpr int AT_BN = 32;        // keys per warp tile
constexpr int AT_WARPS = 4;
constexpr int AT_DH = 128;
constexpr int AT_STAGE_BYTES = 2 * AT_BN * AT_DH * 2;            // K tile + V tile
constexpr int AT_SMEM = AT_WARPS * 2 * AT_STAGE_BYTES + AT_BM * AT_DH * 2 + 1024;

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float* c, const uint32_t* a, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
    const int sz = valid ? 16 : 0;
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sz) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}
// byte offset of 16-byte chunk `ch` of row `row` in a [rows][128] bf16 tile, XOR-swizzled
__device__ __forceinline__ uint32_t sw_off(int row, int ch) { return (uint32_t)(row * 256 + ((ch ^ (row & 7)) << 4)); }

// 2^x by the special-function unit (relative error ~2^-22); scores are kept in the log2 domain so that
// every probability costs one multiply-add and one ex2
__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
constexpr float LOG2E = 1.4426950408889634f;
constexpr float LN2 = 0.6931471805599453f;

struct AttnMmaArgs {
    AttnArgs a;
    int rows_per_seq;   // forward rows per sequence (stand-alone: n_rows)
    int tiles_per_seq;
};

__global__ void __launch_bounds__(AT_WARPS * 32) attention_mma_kernel(AttnMmaArgs g) {
    KERNEL_PROLOGUE(7);   // __launch_bounds__
    extern __shared__ uint8_t at_smem_raw[];
    __shared__ float red_m[AT_WARPS][AT_BM], red_l[AT_WARPS][AT_BM], red_kl[AT_WARPS][AT_BM];
    __shared__ float lse_sh[AT_BM];
    __shared__ float* prev_sh[AT_BM];
    __shared__ int valid_sh[AT_BM];
    const AttnArgs& a = g.a;
    uint8_t* smem = (uint8_t*)(((uintptr_t)at_smem_raw + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int seq = blockIdx.x / g.tiles_per_seq, tile = blockIdx.x - seq * g.tiles_per_seq;
    const int h = blockIdx.y;
    const int g_kv = (h * a.n_kv) / a.n_heads;
    const int dq = a.n_heads * AT_DH, dkv = a.n_kv * AT_DH;
    const int row0 = seq * g.rows_per_seq + tile * AT_BM;
    const int n_in_tile = min(AT_BM, g.rows_per_seq - tile * AT_BM);

    uint8_t* q_s = smem + AT_WARPS * 2 * AT_STAGE_BYTES;
    uint8_t* my_stage = smem + warp * 2 * AT_STAGE_BYTES;
    const uint32_t q_u32 = (uint32_t)__cvta_generic_to_shared(q_s);
    const uint32_t st_u32 = (uint32_t)__cvta_generic_to_shared(my_stage);

    // ---- row bookkeeping + Q tile ----------------------------------------------------------
    int kv_seq = seq;
    if (threadIdx.x < AT_BM) {
        const int i = threadIdx.x;
        float* prev = nullptr;
        int valid = 0;
        if (i < n_in_tile) {
            const int r = row0 + i;
            if (a.rows) {
                const Row rw = a.rows[r];
                if (rw.pos >= 0) {
                    valid = 1;
                    if (rw.widx >= 0 && a.pprev) prev = a.pprev + (((size_t)rw.seq * a.W_max + rw.widx) * a.n_heads + h) * a.N;
                    else if (rw.aidx >= 0 && a.aprev) prev = a.aprev + (((size_t)rw.seq * a.B + rw.aidx) * a.n_heads + h) * a.N;
                }
            } else {
                valid = 1;
                if (a.pprev) prev = a.pprev + ((size_t)r * a.n_heads + h) * a.N;
            }
        }
        prev_sh[i] = prev;
        valid_sh[i] = valid;
    }
    if (!a.rows) kv_seq = 0;
    for (int t = threadIdx.x; t < AT_BM * 16; t += blockDim.x) {
        const int i = t >> 4, ch = t & 15;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (i < n_in_tile) v = *reinterpret_cast<const uint4*>((const __nv_bfloat16*)a.q + (size_t)(row0 + i) * dq + h * AT_DH + ch * 8);
        *reinterpret_cast<uint4*>(q_s + sw_off(i, ch)) = v;
    }
    __syncthreads();
    // invalid rows may hold uninitialised q: zero them so no NaN/Inf enters the tile's arithmetic
    for (int t = threadIdx.x; t < AT_BM * 16; t += blockDim.x) {
        const int i = t >> 4, ch = t & 15;
        if (!valid_sh[i]) *reinterpret_cast<uint4*>(q_s + sw_off(i, ch)) = make_uint4(0, 0, 0, 0);
    }
    __syncthreads();

    uint32_t qf[8][4];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        const int i = lane >> 3, r = lane & 7;
        ldsm_x4(q_u32 + sw_off((i & 1) * 8 + r, 2 * k + (i >> 1)), qf[k][0], qf[k][1], qf[k][2], qf[k][3]);
    }

    const __nv_bfloat16* Kg = (const __nv_bfloat16*)a.kc + (size_t)kv_seq * a.N * dkv + g_kv * AT_DH;
    const __nv_bfloat16* Vg = (const __nv_bfloat16*)a.vc + (size_t)kv_seq * a.N * dkv + g_kv * AT_DH;
    const int n_tiles = (a.N + AT_BN - 1) / AT_BN;
    const int my_tiles = warp < n_tiles ? (n_tiles - warp + AT_WARPS - 1) / AT_WARPS : 0;

    auto load_tile = [&](int t, int stage, bool with_v) {
        const int key0 = t * AT_BN;
        const uint32_t kb = st_u32 + stage * AT_STAGE_BYTES, vb = kb + AT_BN * AT_DH * 2;
        for (int c = lane; c < AT_BN * 16; c += 32) {
            const int r = c >> 4, ch = c & 15;
            const int key = key0 + r;
            const bool ok = key < a.N;
            const size_t off = (size_t)(ok ? key : 0) * dkv + ch * 8;
            cp_async16(kb + sw_off(r, ch), Kg + off, ok);
            if (with_v) cp_async16(vb + sw_off(r, ch), Vg + off, ok);
        }
        cp_async_commit();
    };
    // scores of one 32-key tile: s[nt][0..3], nt = 0..3 (8 keys each)
    auto scores = [&](int stage, float (*s)[4]) {
        const uint32_t kb = st_u32 + stage * AT_STAGE_BYTES;
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) { s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f; }
#pragma unroll
        for (int k = 0; k < 8; ++k) {
#pragma unroll
            for (int np = 0; np < 2; ++np) {
                const int i = lane >> 3, r = lane & 7;
                uint32_t b0, b1, b2, b3;
                ldsm_x4(kb + sw_off((2 * np + (i >> 1)) * 8 + r, 2 * k + (i & 1)), b0, b1, b2, b3);
                mma_bf16(s[2 * np], qf[k], b0, b1);
                mma_bf16(s[2 * np + 1], qf[k], b2, b3);
            }
        }
    };

    const int r_lo = lane >> 2, r_hi = r_lo + 8;
    const int cpair = (lane & 3) * 2;

    // ---- pass 1: log-sum-exp -----------------------------------------------------------------
    float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;
    if (my_tiles > 0) load_tile(warp, 0, false);
    for (int it = 0; it < my_tiles; ++it) {
        const int t = warp + it * AT_WARPS;
        if (it + 1 < my_tiles) { load_tile(t + AT_WARPS, (it + 1) & 1, false); cp_async_wait<1>(); }
        else cp_async_wait<0>();
        __syncwarp();
        float s[4][4];
        scores(it & 1, s);
        float tm_lo = -INFINITY, tm_hi = -INFINITY;
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int key = t * AT_BN + nt * 8 + cpair + e;
                const bool ok = key < a.N;
                s[nt][e] = ok ? s[nt][e] * a.scale : -INFINITY;
                s[nt][2 + e] = ok ? s[nt][2 + e] * a.scale : -INFINITY;
                tm_lo = fmaxf(tm_lo, s[nt][e]);
                tm_hi = fmaxf(tm_hi, s[nt][2 + e]);
            }
        }
        tm_lo = fmaxf(tm_lo, __shfl_xor_sync(0xffffffffu, tm_lo, 1));
        tm_lo = fmaxf(tm_lo, __shfl_xor_sync(0xffffffffu, tm_lo, 2));
        tm_hi = fmaxf(tm_hi, __shfl_xor_sync(0xffffffffu, tm_hi, 1));
        tm_hi = fmaxf(tm_hi, __shfl_xor_sync(0xffffffffu, tm_hi, 2));
        const float nm_lo = fmaxf(m_lo, tm_lo), nm_hi = fmaxf(m_hi, tm_hi);
        float sl = 0.f, sh = 0.f;
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
#pragma unroll
            for (int e = 0; e < 2; ++e) { sl += expf(s[nt][e] - nm_lo); sh += expf(s[nt][2 + e] - nm_hi); }
        }
        sl += __shfl_xor_sync(0xffffffffu, sl, 1); sl += __shfl_xor_sync(0xffffffffu, sl, 2);
        sh += __shfl_xor_sync(0xffffffffu, sh, 1); sh += __shfl_xor_sync(0xffffffffu, sh, 2);
        l_lo = l_lo * expf(m_lo - nm_lo) + sl;
        l_hi = l_hi * expf(m_hi - nm_hi) + sh;
        m_lo = nm_lo; m_hi = nm_hi;
        __syncwarp();
    }
    if ((lane & 3) == 0) {
        red_m[warp][r_lo] = m_lo; red_l[warp][r_lo] = l_lo;
        red_m[warp][r_hi] = m_hi; red_l[warp][r_hi] = l_hi;
    }
    __syncthreads();
    if (threadIdx.x < AT_BM) {
        const int i = threadIdx.x;
        float mx = -INFINITY;
        for (int w = 0; w < AT_WARPS; ++w) mx = fmaxf(mx, red_m[w][i]);
        float sum = 0.f;
        for (int w = 0; w < AT_WARPS; ++w)
            if (red_l[w][i] > 0.f) sum += red_l[w][i] * expf(red_m[w][i] - mx);
        lse_sh[i] = mx + logf(sum);
    }
    __syncthreads();
    const float lse_lo = lse_sh[r_lo], lse_hi = lse_sh[r_hi];
    float* prev_lo = prev_sh[r_lo];
    float* prev_hi = prev_sh[r_hi];

    // ---- pass 2: logp, KL, stored rows, P V ---------------------------------------------------
    float o[16][4];
#pragma unroll
    for (int nt = 0; nt < 16; ++nt) { o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f; }
    float kl_lo = 0.f, kl_hi = 0.f;
    if (my_tiles > 0) load_tile(warp, 0, true);
    for (int it = 0; it < my_tiles; ++it) {
        const int t = warp + it * AT_WARPS;
        if (it + 1 < my_tiles) { load_tile(t + AT_WARPS, (it + 1) & 1, true); cp_async_wait<1>(); }
        else cp_async_wait<0>();
        __syncwarp();
        // stored rows of this tile first: all loads are issued together, before any of the stores below
        float pv_lo[4][2], pv_hi[4][2];
#pragma unroll
        for (int nt = 0; nt < 4; ++nt)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int key = t * AT_BN + nt * 8 + cpair + e;
                pv_lo[nt][e] = (a.record_kl && prev_lo && key < a.N) ? prev_lo[key] : 0.f;
                pv_hi[nt][e] = (a.record_kl && prev_hi && key < a.N) ? prev_hi[key] : 0.f;
            }
        float s[4][4];
        scores(it & 1, s);
        uint32_t pf[2][4];
        float lp_lo[4][2], lp_hi[4][2];
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
            float p[4];
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int key = t * AT_BN + nt * 8 + cpair + e;
                const bool ok = key < a.N;
                lp_lo[nt][e] = s[nt][e] * a.scale - lse_lo; lp_hi[nt][e] = s[nt][2 + e] * a.scale - lse_hi;
                const float p_lo = ok ? fast_exp2(lp_lo[nt][e] * LOG2E) : 0.f, p_hi = ok ? fast_exp2(lp_hi[nt][e] * LOG2E) : 0.f;
                if (ok && a.record_kl) {
                    if (prev_lo) kl_lo += p_lo * (lp_lo[nt][e] - pv_lo[nt][e]);
                    if (prev_hi) kl_hi += p_hi * (lp_hi[nt][e] - pv_hi[nt][e]);
                }
                p[e] = p_lo; p[2 + e] = p_hi;
            }
            pf[nt >> 1][(nt & 1) * 2 + 0] = pack_bf16(p[0], p[1]);
            pf[nt >> 1][(nt & 1) * 2 + 1] = pack_bf16(p[2], p[3]);
        }
#pragma unroll
        for (int nt = 0; nt < 4; ++nt)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int key = t * AT_BN + nt * 8 + cpair + e;
                if (prev_lo && key < a.N) prev_lo[key] = lp_lo[nt][e];
                if (prev_hi && key < a.N) prev_hi[key] = lp_hi[nt][e];
            }
        if (a.out) {
            const uint32_t vb = st_u32 + (it & 1) * AT_STAGE_BYTES + AT_BN * AT_DH * 2;
#pragma unroll
            for (int ks = 0; ks < 2; ++ks) {
#pragma unroll
                for (int dp = 0; dp < 8; ++dp) {
                    const int i = lane >> 3, r = lane & 7;
                    uint32_t b0, b1, b2, b3;
                    ldsm_x4_t(vb + sw_off(ks * 16 + (i & 1) * 8 + r, 2 * dp + (i >> 1)), b0, b1, b2, b3);
                    mma_bf16(o[2 * dp], pf[ks], b0, b1);
                    mma_bf16(o[2 * dp + 1], pf[ks], b2, b3);
                }
            }
        }
        __syncwarp();
    }
    // ---- combine the warps' partial results (fixed order) ---------------------------------------
    kl_lo += __shfl_xor_sync(0xffffffffu, kl_lo, 1); kl_lo += __shfl_xor_sync(0xffffffffu, kl_lo, 2);
    kl_hi += __shfl_xor_sync(0xffffffffu, kl_hi, 1); kl_hi += __shfl_xor_sync(0xffffffffu, kl_hi, 2);
    if ((lane & 3) == 0) { red_kl[warp][r_lo] = kl_lo; red_kl[warp][r_hi] = kl_hi; }
    __syncthreads();       // every warp is done with its K/V stages: reuse them for the O partials
    float* o_s = reinterpret_cast<float*>(smem);     // [warps][16][128] fp32 = 32 KB
    if (a.out) {
#pragma unroll
        for (int nt = 0; nt < 16; ++nt) {
            const int col = nt * 8 + cpair;
            float* b0 = o_s + ((size_t)warp * AT_BM + r_lo) * AT_DH + col;
            float* b1 = o_s + ((size_t)warp * AT_BM + r_hi) * AT_DH + col;
            b0[0] = o[nt][0]; b0[1] = o[nt][1]; b1[0] = o[nt][2]; b1[1] = o[nt][3];
        }
    }
    __syncthreads();
    if (a.out) {
        for (int t = threadIdx.x; t < AT_BM * AT_DH / 2; t += blockDim.x) {
            const int i = t / (AT_DH / 2), c = (t % (AT_DH / 2)) * 2;
            if (!valid_sh[i]) continue;
            float v0 = 0.f, v1 = 0.f;
#pragma unroll
            for (int w = 0; w < AT_WARPS; ++w) {
                v0 += o_s[((size_t)w * AT_BM + i) * AT_DH + c];
                v1 += o_s[((size_t)w * AT_BM + i) * AT_DH + c + 1];
            }
            *reinterpret_cast<__nv_bfloat162*>((__nv_bfloat16*)a.out + (size_t)(row0 + i) * dq + h * AT_DH + c) =
                __floats2bfloat162_rn(v0, v1);
        }
    }
    if (a.kl && threadIdx.x < AT_BM && valid_sh[threadIdx.x]) {
        const int i = threadIdx.x;
        float kl = 0.f;
        for (int w = 0; w < AT_WARPS; ++w) kl += red_kl[w][i];
        a.kl[(size_t)(row0 + i) * a.n_heads + h] = (prev_sh[i] && a.record_kl) ? kl : 0.f;
    }
}

// ------------------------------------------------------------------------------------------
// Single-pass variant for N <= NW * TPW * 32 keys: every warp keeps the scores of its (at most
// TPW) key tiles in registers, so K is read once.  Loads of a warp form one sequence
// K_0 .. K_{n-1}, V_0 .. V_{n-1} through a private two-slot ring; the V tiles stream in while
// the warps exchange their row maxima / sums.  Stored rows are read before they are rewritten,
// a tile at a time, with all loads of the tile issued together.
// ------------------------------------------------------------------------------------------
constexpr int SP_SLOT_BYTES = AT_BN * AT_DH * 2;     // one K or V tile: 8 KB

// CL = 2: the keys of one (row tile, head) are split over a cluster of two CTAs (few rows: more SMs pull K/V,
// and each warp's K and V tile are all in flight from the start).  The two CTAs exchange their rows'
// (max, sum), partial KL and partial outputs through distributed shared memory; rank 0 writes the results.
template <int NW, int TPW, int CL>
__global__ void __launch_bounds__(NW * 32) attention_sp_kernel(AttnMmaArgs g) {
    pdl_trigger();        // (the wait for the kernel before this one comes after the first loads of untouched key tiles)
    extern __shared__ uint8_t at_smem_raw[];
    __shared__ float red_m[NW][AT_BM], red_l[NW][AT_BM], red_kl[NW][AT_BM];
    __shared__ float lse_sh[AT_BM];
    __shared__ float* prev_sh[AT_BM];
    __shared__ int valid_sh[AT_BM];
    __shared__ float2 cl_ml[AT_BM];       // CL = 2: this CTA's (max, sum) per row
    __shared__ float cl_kl[AT_BM];
    const AttnArgs& a = g.a;
    uint8_t* smem = (uint8_t*)(((uintptr_t)at_smem_raw + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rank = CL > 1 ? (int)cluster_rank() : 0;
    const int bx = CL > 1 ? blockIdx.x / CL : blockIdx.x;
    const int seq = bx / g.tiles_per_seq, tile = bx - seq * g.tiles_per_seq;
    const int h = blockIdx.y;
    const int g_kv = (h * a.n_kv) / a.n_heads;
    const int dq = a.n_heads * AT_DH, dkv = a.n_kv * AT_DH;
    const int row0 = seq * g.rows_per_seq + tile * AT_BM;
    const int n_in_tile = min(AT_BM, g.rows_per_seq - tile * AT_BM);

    uint8_t* q_s = smem + NW * 2 * SP_SLOT_BYTES;
    const uint32_t q_u32 = (uint32_t)__cvta_generic_to_shared(q_s);
    const uint32_t ring = (uint32_t)__cvta_generic_to_shared(smem + warp * 2 * SP_SLOT_BYTES);

    const int kv_seq = a.rows ? seq : 0;
    const __nv_bfloat16* Kg = (const __nv_bfloat16*)a.kc + (size_t)kv_seq * a.N * dkv + g_kv * AT_DH;
    const __nv_bfloat16* Vg = (const __nv_bfloat16*)a.vc + (size_t)kv_seq * a.N * dkv + g_kv * AT_DH;
    const int n_tiles = (a.N + AT_BN - 1) / AT_BN;
    // key tile of (warp, i): warp + (i * CL + rank) * NW
    int my_tiles = 0;
#pragma unroll
    for (int i = 0; i < TPW; ++i) my_tiles += (warp + (i * CL + rank) * NW < n_tiles) ? 1 : 0;
    const int n_loads = a.out ? 2 * my_tiles : my_tiles;

    auto issue = [&](int j) {      // load j of this warp's sequence into slot j & 1
        const bool is_v = j >= my_tiles;
        const int t = warp + ((is_v ? j - my_tiles : j) * CL + rank) * NW;
        const __nv_bfloat16* src = is_v ? Vg : Kg;
        const uint32_t dst = ring + (j & 1) * SP_SLOT_BYTES;
        const int key0 = t * AT_BN;
#pragma unroll 4
        for (int c = lane; c < AT_BN * 16; c += 32) {
            const int r = c >> 4, ch = c & 15;
            const int key = key0 + r;
            const bool ok = key < a.N;
            cp_async16(dst + sw_off(r, ch), src + (size_t)(ok ? key : 0) * dkv + ch * 8, ok);
        }
        cp_async_commit();
    };
    // Key tiles outside [dirty_lo, dirty_hi) were last written by an earlier forward, which the host has waited for:
    // their K / V can be on their way while the projection before this kernel still runs.  q, the row table and
    // the rows that projection writes come after the wait.
    auto load_clean = [&](int j) {
        const bool is_v = j >= my_tiles;
        const int lo = (warp + ((is_v ? j - my_tiles : j) * CL + rank) * NW) * AT_BN;
        return lo + AT_BN <= a.dirty_lo || lo >= a.dirty_hi;
    };
    int issued = 0;
    if (n_loads > 0 && load_clean(0)) {
        issue(0);
        issued = 1;
        if (n_loads > 1 && load_clean(1)) { issue(1); issued = 2; }
    }
    pdl_wait();
    trace_stamp(7);
    if (issued < 1 && n_loads > 0) issue(0);
    if (issued < 2 && n_loads > 1) issue(1);

    // ---- row bookkeeping + Q tile (overlap the first K loads; neither waits for the other) ----------
    // Rows without a valid descriptor may hold stale q values: they only ever affect their own row of
    // the tile, which is never written.
    for (int t = threadIdx.x; t < AT_BM * 16; t += blockDim.x) {
        const int i = t >> 4, ch = t & 15;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (i < n_in_tile) v = *reinterpret_cast<const uint4*>((const __nv_bfloat16*)a.q + (size_t)(row0 + i) * dq + h * AT_DH + ch * 8);
        *reinterpret_cast<uint4*>(q_s + sw_off(i, ch)) = v;
    }
    if (threadIdx.x < AT_BM) {
        const int i = threadIdx.x;
        float* prev = nullptr;
        int valid = 0;
        if (i < n_in_tile) {
            const int r = row0 + i;
            if (a.rows) {
                const Row rw = a.rows[r];
                if (rw.pos >= 0) {
                    valid = 1;
                    if (rw.widx >= 0 && a.pprev) prev = a.pprev + (((size_t)rw.seq * a.W_max + rw.widx) * a.n_heads + h) * a.N;
                    else if (rw.aidx >= 0 && a.aprev) prev = a.aprev + (((size_t)rw.seq * a.B + rw.aidx) * a.n_heads + h) * a.N;
                }
            } else {
                valid = 1;
                if (a.pprev) prev = a.pprev + ((size_t)r * a.n_heads + h) * a.N;
            }
        }
        prev_sh[i] = prev;
        valid_sh[i] = valid;
    }
    __syncthreads();
    uint32_t qf[8][4];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        const int i = lane >> 3, r = lane & 7;
        ldsm_x4(q_u32 + sw_off((i & 1) * 8 + r, 2 * k + (i >> 1)), qf[k][0], qf[k][1], qf[k][2], qf[k][3]);
    }

    const int r_lo = lane >> 2, r_hi = r_lo + 8;
    const int cpair = (lane & 3) * 2;

    // ---- scores of my tiles, kept in registers ---------------------------------------------------
    const float scale2 = a.scale * LOG2E;
    float s[TPW][4][4];
    float m_lo = -INFINITY, m_hi = -INFINITY;
#pragma unroll
    for (int i = 0; i < TPW; ++i) {
        if (i < my_tiles) {
            if (i + 1 < n_loads) cp_async_wait<1>(); else cp_async_wait<0>();
            __syncwarp();
            const uint32_t kb = ring + (i & 1) * SP_SLOT_BYTES;
#pragma unroll
            for (int nt = 0; nt < 4; ++nt) { s[i][nt][0] = s[i][nt][1] = s[i][nt][2] = s[i][nt][3] = 0.f; }
#pragma unroll
            for (int k = 0; k < 8; ++k) {
#pragma unroll
                for (int np = 0; np < 2; ++np) {
                    const int ii = lane >> 3, r = lane & 7;
                    uint32_t b0, b1, b2, b3;
                    ldsm_x4(kb + sw_off((2 * np + (ii >> 1)) * 8 + r, 2 * k + (ii & 1)), b0, b1, b2, b3);
                    mma_bf16(s[i][2 * np], qf[k], b0, b1);
                    mma_bf16(s[i][2 * np + 1], qf[k], b2, b3);
                }
            }
            __syncwarp();
            if (i + 2 < n_loads) issue(i + 2);
            const int t = warp + (i * CL + rank) * NW;
#pragma unroll
            for (int nt = 0; nt < 4; ++nt) {
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const bool ok = t * AT_BN + nt * 8 + cpair + e < a.N;
                    s[i][nt][e] = ok ? s[i][nt][e] * scale2 : -INFINITY;          // log2 domain
                    s[i][nt][2 + e] = ok ? s[i][nt][2 + e] * scale2 : -INFINITY;
                    m_lo = fmaxf(m_lo, s[i][nt][e]);
                    m_hi = fmaxf(m_hi, s[i][nt][2 + e]);
                }
            }
        }
    }
    m_lo = fmaxf(m_lo, __shfl_xor_sync(0xffffffffu, m_lo, 1));
    m_lo = fmaxf(m_lo, __shfl_xor_sync(0xffffffffu, m_lo, 2));
    m_hi = fmaxf(m_hi, __shfl_xor_sync(0xffffffffu, m_hi, 1));
    m_hi = fmaxf(m_hi, __shfl_xor_sync(0xffffffffu, m_hi, 2));
    float l_lo = 0.f, l_hi = 0.f;
#pragma unroll
    for (int i = 0; i < TPW; ++i) {
        if (i < my_tiles) {
#pragma unroll
            for (int nt = 0; nt < 4; ++nt)
#pragma unroll
                for (int e = 0; e < 2; ++e) { l_lo += fast_exp2(s[i][nt][e] - m_lo); l_hi += fast_exp2(s[i][nt][2 + e] - m_hi); }
        }
    }
    l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1); l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
    l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1); l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
    if ((lane & 3) == 0) {
        red_m[warp][r_lo] = m_lo; red_l[warp][r_lo] = my_tiles ? l_lo : 0.f;
        red_m[warp][r_hi] = m_hi; red_l[warp][r_hi] = my_tiles ? l_hi : 0.f;
    }
    __syncthreads();
    if (threadIdx.x < AT_BM) {
        const int i = threadIdx.x;
        float mx = -INFINITY;
        for (int w = 0; w < NW; ++w) mx = fmaxf(mx, red_m[w][i]);
        float sum = 0.f;
        for (int w = 0; w < NW; ++w)
            if (red_l[w][i] > 0.f) sum += red_l[w][i] * fast_exp2(red_m[w][i] - mx);
        if (CL > 1) cl_ml[i] = make_float2(mx, sum);
        else lse_sh[i] = mx + log2f(sum);       // log2 domain
    }
    if (CL > 1) {
        cluster_sync_all();
        if (threadIdx.x < AT_BM) {
            // both CTAs combine the two halves in rank order, so both get the same value
            const int i = threadIdx.x;
            const uint32_t mine = (uint32_t)__cvta_generic_to_shared(&cl_ml[i]);
            const float2 h0 = ld_dsmem_f2(dsmem_addr(mine, 0)), h1 = ld_dsmem_f2(dsmem_addr(mine, 1));
            const float mx = fmaxf(h0.x, h1.x);
            float sum = 0.f;
            if (h0.y > 0.f) sum += h0.y * fast_exp2(h0.x - mx);
            if (h1.y > 0.f) sum += h1.y * fast_exp2(h1.x - mx);
            lse_sh[i] = mx + log2f(sum);
        }
    }
    __syncthreads();
    const float lse_lo = lse_sh[r_lo], lse_hi = lse_sh[r_hi];
    float* prev_lo = prev_sh[r_lo];
    float* prev_hi = prev_sh[r_hi];
    const bool vec = (a.N & 1) == 0;

    // ---- logp, KL, stored rows, P V ----------------------------------------------------------------
    float o[16][4];
#pragma unroll
    for (int nt = 0; nt < 16; ++nt) { o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f; }
    float kl_lo = 0.f, kl_hi = 0.f;
#pragma unroll
    for (int i = 0; i < TPW; ++i) {
        if (i < my_tiles) {
            const int t = warp + (i * CL + rank) * NW;
            // stored rows of this tile: all loads first
            float pv_lo[4][2], pv_hi[4][2];
#pragma unroll
            for (int nt = 0; nt < 4; ++nt) {
                const int key = t * AT_BN + nt * 8 + cpair;
                pv_lo[nt][0] = pv_lo[nt][1] = pv_hi[nt][0] = pv_hi[nt][1] = 0.f;
                if (a.record_kl) {
                    if (vec) {
                        if (prev_lo && key < a.N) { const float2 v = *reinterpret_cast<const float2*>(prev_lo + key); pv_lo[nt][0] = v.x; pv_lo[nt][1] = v.y; }
                        if (prev_hi && key < a.N) { const float2 v = *reinterpret_cast<const float2*>(prev_hi + key); pv_hi[nt][0] = v.x; pv_hi[nt][1] = v.y; }
                    } else {
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            if (prev_lo && key + e < a.N) pv_lo[nt][e] = prev_lo[key + e];
                            if (prev_hi && key + e < a.N) pv_hi[nt][e] = prev_hi[key + e];
                        }
                    }
                }
            }
            uint32_t pf[2][4];
            float lp_lo[4][2], lp_hi[4][2];
#pragma unroll
            for (int nt = 0; nt < 4; ++nt) {
                float p[4];
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const bool ok = t * AT_BN + nt * 8 + cpair + e < a.N;
                    const float d_lo = s[i][nt][e] - lse_lo, d_hi = s[i][nt][2 + e] - lse_hi;
                    const float p_lo = ok ? fast_exp2(d_lo) : 0.f, p_hi = ok ? fast_exp2(d_hi) : 0.f;
                    lp_lo[nt][e] = d_lo * LN2; lp_hi[nt][e] = d_hi * LN2;       // natural-log probabilities
                    if (ok && a.record_kl) {
                        if (prev_lo) kl_lo += p_lo * (lp_lo[nt][e] - pv_lo[nt][e]);
                        if (prev_hi) kl_hi += p_hi * (lp_hi[nt][e] - pv_hi[nt][e]);
                    }
                    p[e] = p_lo; p[2 + e] = p_hi;
                }
                pf[nt >> 1][(nt & 1) * 2 + 0] = pack_bf16(p[0], p[1]);
                pf[nt >> 1][(nt & 1) * 2 + 1] = pack_bf16(p[2], p[3]);
            }
#pragma unroll
            for (int nt = 0; nt < 4; ++nt) {
                const int key = t * AT_BN + nt * 8 + cpair;
                if (vec) {
                    if (prev_lo && key < a.N) *reinterpret_cast<float2*>(prev_lo + key) = make_float2(lp_lo[nt][0], lp_lo[nt][1]);
                    if (prev_hi && key < a.N) *reinterpret_cast<float2*>(prev_hi + key) = make_float2(lp_hi[nt][0], lp_hi[nt][1]);
                } else {
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        if (prev_lo && key + e < a.N) prev_lo[key + e] = lp_lo[nt][e];
                        if (prev_hi && key + e < a.N) prev_hi[key + e] = lp_hi[nt][e];
                    }
                }
            }
            if (a.out) {
                const int j = my_tiles + i;
                if (j + 1 < n_loads) cp_async_wait<1>(); else cp_async_wait<0>();
                __syncwarp();
                const uint32_t vb = ring + (j & 1) * SP_SLOT_BYTES;
#pragma unroll
                for (int ks = 0; ks < 2; ++ks) {
#pragma unroll
                    for (int dp = 0; dp < 8; ++dp) {
                        const int ii = lane >> 3, r = lane & 7;
                        uint32_t b0, b1, b2, b3;
                        ldsm_x4_t(vb + sw_off(ks * 16 + (ii & 1) * 8 + r, 2 * dp + (ii >> 1)), b0, b1, b2, b3);
                        mma_bf16(o[2 * dp], pf[ks], b0, b1);
                        mma_bf16(o[2 * dp + 1], pf[ks], b2, b3);
                    }
                }
                __syncwarp();
                if (j + 2 < n_loads) issue(j + 2);
            }
        }
    }
    // ---- combine the warps' partial results (fixed order) ---------------------------------------
    kl_lo += __shfl_xor_sync(0xffffffffu, kl_lo, 1); kl_lo += __shfl_xor_sync(0xffffffffu, kl_lo, 2);
    kl_hi += __shfl_xor_sync(0xffffffffu, kl_hi, 1); kl_hi += __shfl_xor_sync(0xffffffffu, kl_hi, 2);
    if ((lane & 3) == 0) { red_kl[warp][r_lo] = kl_lo; red_kl[warp][r_hi] = kl_hi; }
    __syncthreads();       // every warp is done with its ring: reuse it for the O partials
    float* o_s = reinterpret_cast<float*>(smem);     // [NW][16][128] fp32 = NW * 8 KB <= ring size
    if (a.out) {
#pragma unroll
        for (int nt = 0; nt < 16; ++nt) {
            const int col = nt * 8 + cpair;
            *reinterpret_cast<float2*>(o_s + ((size_t)warp * AT_BM + r_lo) * AT_DH + col) = make_float2(o[nt][0], o[nt][1]);
            *reinterpret_cast<float2*>(o_s + ((size_t)warp * AT_BM + r_hi) * AT_DH + col) = make_float2(o[nt][2], o[nt][3]);
        }
    }
    __syncthreads();
    float* o_red = reinterpret_cast<float*>(smem + NW * 2 * SP_SLOT_BYTES + AT_BM * AT_DH * 2);   // CL = 2: [16][128] fp32
    if (CL > 1) {
        // each CTA adds up its warps; rank 0 then adds the two CTAs (rank order) and writes
        if (a.out) {
            for (int t = threadIdx.x; t < AT_BM * AT_DH / 2; t += blockDim.x) {
                const int i = t / (AT_DH / 2), c = (t % (AT_DH / 2)) * 2;
                float v0 = 0.f, v1 = 0.f;
#pragma unroll
                for (int w = 0; w < NW; ++w) {
                    const float2 v = *reinterpret_cast<const float2*>(o_s + ((size_t)w * AT_BM + i) * AT_DH + c);
                    v0 += v.x; v1 += v.y;
                }
                *reinterpret_cast<float2*>(o_red + i * AT_DH + c) = make_float2(v0, v1);
            }
        }
        if (threadIdx.x < AT_BM) {
            float kl = 0.f;
            for (int w = 0; w < NW; ++w) kl += red_kl[w][threadIdx.x];
            cl_kl[threadIdx.x] = kl;
        }
        cluster_sync_all();
        if (rank == 0) {
            if (a.out) {
                const uint32_t peer = dsmem_addr((uint32_t)__cvta_generic_to_shared(o_red), 1);
                for (int t = threadIdx.x; t < AT_BM * AT_DH / 2; t += blockDim.x) {
                    const int i = t / (AT_DH / 2), c = (t % (AT_DH / 2)) * 2;
                    if (!valid_sh[i]) continue;
                    const float2 v0 = *reinterpret_cast<const float2*>(o_red + i * AT_DH + c);
                    const float2 v1 = ld_dsmem_f2(peer + (uint32_t)((i * AT_DH + c) * 4));
                    *reinterpret_cast<__nv_bfloat162*>((__nv_bfloat16*)a.out + (size_t)(row0 + i) * dq + h * AT_DH + c) =
                        __floats2bfloat162_rn(v0.x + v1.x, v0.y + v1.y);
                }
            }
            if (a.kl && threadIdx.x < AT_BM && valid_sh[threadIdx.x]) {
                const int i = threadIdx.x;
                float other;
                asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(other)
                             : "r"(dsmem_addr((uint32_t)__cvta_generic_to_shared(&cl_kl[i]), 1)) : "memory");
                a.kl[(size_t)(row0 + i) * a.n_heads + h] = (prev_sh[i] && a.record_kl) ? cl_kl[i] + other : 0.f;
            }
        }
        cluster_sync_all();       // rank 1 stays until rank 0 has read its shared memory
        return;
    }
    if (a.out) {
        for (int t = threadIdx.x; t < AT_BM * AT_DH / 2; t += blockDim.x) {
            const int i = t / (AT_DH / 2), c = (t % (AT_DH / 2)) * 2;
            if (!valid_sh[i]) continue;
            float v0 = 0.f, v1 = 0.f;
#pragma unroll
            for (int w = 0; w < NW; ++w) {
                const float2 v = *reinterpret_cast<const float2*>(o_s + ((size_t)w * AT_BM + i) * AT_DH + c);
                v0 += v.x; v1 += v.y;
            }
            *reinterpret_cast<__nv_bfloat162*>((__nv_bfloat16*)a.out + (size_t)(row0 + i) * dq + h * AT_DH + c) =
                __floats2bfloat162_rn(v0, v1);
        }
    }
    if (a.kl && threadIdx.x < AT_BM && valid_sh[threadIdx.x]) {
        const int i = threadIdx.x;
        float kl = 0.f;
        for (int w = 0; w < NW; ++w) kl += red_kl[w][i];
        a.kl[(size_t)(row0 + i) * a.n_heads + h] = (prev_sh[i] && a.record_kl) ? kl : 0.f;
    }
}

// ------------------------------------------------------------------------------------------
// Many-rows variant (block-entry forwards, long sequences, batches): one CTA = 64 query rows of one
// head, 4 warps x 16 rows; every 64-key K/V tile is staged once per CTA in shared memory (cp.async
// ring) and used by all four warps, so K/V are re-read once per 64 rows instead of once per
// 16.  Each warp keeps its rows' running max / sum and output accumulator in registers; no cross-warp
// reduction is needed.
// ------------------------------------------------------------------------------------------
constexpr int BG_BM = 64, BG_BN = 64, BG_WARPS = 4, BG_STAGES = 3;
constexpr int BG_TILE_BYTES = BG_BN * AT_DH * 2;                  // 16 KB: one K or V tile
constexpr int BG_SMEM = BG_STAGES * 2 * BG_TILE_BYTES + 1024;     // 97 KB: two CTAs per SM

__device__ __forceinline__ void cp_async_wait_pending(int n) {    // at most n groups still in flight
    if (n <= 0) cp_async_wait<0>();
    else if (n == 1) cp_async_wait<1>();
    else cp_async_wait<2>();
}

// K/V tiles go through a three-stage cp.async ring (two tiles ahead of the one being used); the Q tile
// borrows the third stage until its fragments are in registers.  When no row of the launch records
// attention rows (no stored rows, no KL) the kernel makes ONE pass with a running maximum: the output
// accumulator is rescaled when the maximum grows and divided by the row sum at the end, so K is read
// once.  Otherwise two passes (exact log-probabilities need the final row sum before anything is stored).
__global__ void __launch_bounds__(BG_WARPS * 32) attention_big_kernel(AttnMmaArgs g) {
    KERNEL_PROLOGUE(7);
    extern __shared__ uint8_t at_smem_raw[];
    __shared__ float* prev_sh[BG_BM];
    __shared__ int valid_sh[BG_BM];
    const AttnArgs& a = g.a;
    uint8_t* smem = (uint8_t*)(((uintptr_t)at_smem_raw + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int seq = blockIdx.x / g.tiles_per_seq, tile = blockIdx.x - seq * g.tiles_per_seq;   // 64-row tiles here
    const int h = blockIdx.y;
    const int g_kv = (h * a.n_kv) / a.n_heads;
    const int dq = a.n_heads * AT_DH, dkv = a.n_kv * AT_DH;
    const int row0 = seq * g.rows_per_seq + tile * BG_BM;
    const int n_in_tile = min(BG_BM, g.rows_per_seq - tile * BG_BM);
    const uint32_t st_u32 = (uint32_t)__cvta_generic_to_shared(smem);
    uint8_t* q_s = smem + (BG_STAGES - 1) * 2 * BG_TILE_BYTES;       // borrowed: the last stage's K slot
    const uint32_t q_u32 = (uint32_t)__cvta_generic_to_shared(q_s);
    const int kv_seq = a.rows ? seq : 0;
    const __nv_bfloat16* Kg = (const __nv_bfloat16*)a.kc + (size_t)kv_seq * a.N * dkv + g_kv * AT_DH;
    const __nv_bfloat16* Vg = (const __nv_bfloat16*)a.vc + (size_t)kv_seq * a.N * dkv + g_kv * AT_DH;
    const int n_tiles = (a.N + BG_BN - 1) / BG_BN;
    const bool record = (a.pprev != nullptr) || (a.aprev != nullptr);
    const bool single = !record;

    auto load_tile = [&](int t, bool with_v) {
        const int key0 = t * BG_BN;
        const uint32_t kb = st_u32 + (t % BG_STAGES) * 2 * BG_TILE_BYTES, vb = kb + BG_TILE_BYTES;
        for (int c = threadIdx.x; c < BG_BN * 16; c += BG_WARPS * 32) {
            const int r = c >> 4, ch = c & 15;
            const int key = key0 + r;
            const bool ok = key < a.N;
            const size_t off = (size_t)(ok ? key : 0) * dkv + ch * 8;
            cp_async16(kb + sw_off(r, ch), Kg + off, ok);
            if (with_v) cp_async16(vb + sw_off(r, ch), Vg + off, ok);
        }
        cp_async_commit();
    };
    // first pass of the ring: tiles 0 and 1 now, tile 2 once Q has left its stage
    const bool v_first = single && a.out != nullptr;
    load_tile(0, v_first);
    if (n_tiles > 1) load_tile(1, v_first);
    for (int t = threadIdx.x; t < BG_BM * 16; t += blockDim.x) {
        const int i = t >> 4, ch = t & 15;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (i < n_in_tile) v = *reinterpret_cast<const uint4*>((const __nv_bfloat16*)a.q + (size_t)(row0 + i) * dq + h * AT_DH + ch * 8);
        *reinterpret_cast<uint4*>(q_s + sw_off(i, ch)) = v;
    }
    if (threadIdx.x < BG_BM) {
        const int i = threadIdx.x;
        float* prev = nullptr;
        int valid = 0;
        if (i < n_in_tile) {
            const int r = row0 + i;
            if (a.rows) {
                const Row rw = a.rows[r];
                if (rw.pos >= 0) {
                    valid = 1;
                    if (rw.widx >= 0 && a.pprev) prev = a.pprev + (((size_t)rw.seq * a.W_max + rw.widx) * a.n_heads + h) * a.N;
                    else if (rw.aidx >= 0 && a.aprev) prev = a.aprev + (((size_t)rw.seq * a.B + rw.aidx) * a.n_heads + h) * a.N;
                }
            } else {
                valid = 1;
                if (a.pprev) prev = a.pprev + ((size_t)r * a.n_heads + h) * a.N;
            }
        }
        prev_sh[i] = prev;
        valid_sh[i] = valid;
    }
    __syncthreads();
    uint32_t qf[8][4];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        const int i = lane >> 3, r = lane & 7;
        ldsm_x4(q_u32 + sw_off(warp * 16 + (i & 1) * 8 + r, 2 * k + (i >> 1)), qf[k][0], qf[k][1], qf[k][2], qf[k][3]);
    }
    __syncthreads();                                    // Q is in registers: its stage joins the ring
    if (n_tiles > 2) load_tile(2, v_first);
    const int r_lo = warp * 16 + (lane >> 2), r_hi = r_lo + 8;
    const int cpair = (lane & 3) * 2;
    const float scale2 = a.scale * LOG2E;

    auto scores = [&](int t, float (*s)[4]) {     // s[8][4]: 16 rows x 64 keys per warp, raw q.k
        const uint32_t kb = st_u32 + (t % BG_STAGES) * 2 * BG_TILE_BYTES;
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) { s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f; }
#pragma unroll
        for (int k = 0; k < 8; ++k) {
#pragma unroll
            for (int np = 0; np < 4; ++np) {
                const int i = lane >> 3, r = lane & 7;
                uint32_t b0, b1, b2, b3;
                ldsm_x4(kb + sw_off((2 * np + (i >> 1)) * 8 + r, 2 * k + (i & 1)), b0, b1, b2, b3);
                mma_bf16(s[2 * np], qf[k], b0, b1);
                mma_bf16(s[2 * np + 1], qf[k], b2, b3);
            }
        }
    };
    auto pv = [&](int t, const uint32_t (*pf)[4], float (*o)[4]) {      // o += P V for the 64 keys of tile t
        const uint32_t vb = st_u32 + (t % BG_STAGES) * 2 * BG_TILE_BYTES + BG_TILE_BYTES;
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
#pragma unroll
            for (int dp = 0; dp < 8; ++dp) {
                const int i = lane >> 3, r = lane & 7;
                uint32_t b0, b1, b2, b3;
                ldsm_x4_t(vb + sw_off(ks * 16 + (i & 1) * 8 + r, 2 * dp + (i >> 1)), b0, b1, b2, b3);
                mma_bf16(o[2 * dp], pf[ks], b0, b1);
                mma_bf16(o[2 * dp + 1], pf[ks], b2, b3);
            }
        }
    };
    // one step of the ring: request tile t + 2 (its stage was released at the end of step t - 1), wait for tile t
    auto ring_step = [&](int t, bool with_v) {
        if (t >= 1 && t + 2 < n_tiles) load_tile(t + 2, with_v);
        cp_async_wait_pending(min(2, n_tiles - 1 - t));
        __syncthreads();
    };

    float o[16][4];
#pragma unroll
    for (int nt = 0; nt < 16; ++nt) { o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f; }
    float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;
    float kl_lo = 0.f, kl_hi = 0.f;
    float* prev_lo = prev_sh[r_lo];
    float* prev_hi = prev_sh[r_hi];

    if (single) {
        // ---- one pass: running maximum, rescaled accumulator ---------------------------------------------
        for (int t = 0; t < n_tiles; ++t) {
            ring_step(t, a.out != nullptr);
            float s[8][4];
            scores(t, s);
            float tm_lo = -INFINITY, tm_hi = -INFINITY;
#pragma unroll
            for (int nt = 0; nt < 8; ++nt)
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const bool ok = t * BG_BN + nt * 8 + cpair + e < a.N;
                    s[nt][e] = ok ? s[nt][e] * scale2 : -INFINITY;
                    s[nt][2 + e] = ok ? s[nt][2 + e] * scale2 : -INFINITY;
                    tm_lo = fmaxf(tm_lo, s[nt][e]); tm_hi = fmaxf(tm_hi, s[nt][2 + e]);
                }
            tm_lo = fmaxf(tm_lo, __shfl_xor_sync(0xffffffffu, tm_lo, 1)); tm_lo = fmaxf(tm_lo, __shfl_xor_sync(0xffffffffu, tm_lo, 2));
            tm_hi = fmaxf(tm_hi, __shfl_xor_sync(0xffffffffu, tm_hi, 1)); tm_hi = fmaxf(tm_hi, __shfl_xor_sync(0xffffffffu, tm_hi, 2));
            const float nm_lo = fmaxf(m_lo, tm_lo), nm_hi = fmaxf(m_hi, tm_hi);
            const float al_lo = fast_exp2(m_lo - nm_lo), al_hi = fast_exp2(m_hi - nm_hi);
            uint32_t pf[4][4];
            float sl = 0.f, sh = 0.f;
#pragma unroll
            for (int nt = 0; nt < 8; ++nt) {
                float p[4];
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    p[e] = fast_exp2(s[nt][e] - nm_lo); p[2 + e] = fast_exp2(s[nt][2 + e] - nm_hi);
                    sl += p[e]; sh += p[2 + e];
                }
                pf[nt >> 1][(nt & 1) * 2 + 0] = pack_bf16(p[0], p[1]);
                pf[nt >> 1][(nt & 1) * 2 + 1] = pack_bf16(p[2], p[3]);
            }
            l_lo = l_lo * al_lo + sl; l_hi = l_hi * al_hi + sh;
            m_lo = nm_lo; m_hi = nm_hi;
            if (a.out) {
#pragma unroll
                for (int nt = 0; nt < 16; ++nt) { o[nt][0] *= al_lo; o[nt][1] *= al_lo; o[nt][2] *= al_hi; o[nt][3] *= al_hi; }
                pv(t, pf, o);
            }
            __syncthreads();
        }
        l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1); l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
        l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1); l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
        const float il_lo = 1.f / l_lo, il_hi = 1.f / l_hi;
#pragma unroll
        for (int nt = 0; nt < 16; ++nt) { o[nt][0] *= il_lo; o[nt][1] *= il_lo; o[nt][2] *= il_hi; o[nt][3] *= il_hi; }
    } else {
        // ---- pass 1: running max and sum (log2 domain) ---------------------------------------------------
        for (int t = 0; t < n_tiles; ++t) {
            ring_step(t, false);
            float s[8][4];
            scores(t, s);
            float tm_lo = -INFINITY, tm_hi = -INFINITY;
#pragma unroll
            for (int nt = 0; nt < 8; ++nt)
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const bool ok = t * BG_BN + nt * 8 + cpair + e < a.N;
                    s[nt][e] = ok ? s[nt][e] * scale2 : -INFINITY;
                    s[nt][2 + e] = ok ? s[nt][2 + e] * scale2 : -INFINITY;
                    tm_lo = fmaxf(tm_lo, s[nt][e]); tm_hi = fmaxf(tm_hi, s[nt][2 + e]);
                }
            tm_lo = fmaxf(tm_lo, __shfl_xor_sync(0xffffffffu, tm_lo, 1)); tm_lo = fmaxf(tm_lo, __shfl_xor_sync(0xffffffffu, tm_lo, 2));
            tm_hi = fmaxf(tm_hi, __shfl_xor_sync(0xffffffffu, tm_hi, 1)); tm_hi = fmaxf(tm_hi, __shfl_xor_sync(0xffffffffu, tm_hi, 2));
            const float nm_lo = fmaxf(m_lo, tm_lo), nm_hi = fmaxf(m_hi, tm_hi);
            float sl = 0.f, sh = 0.f;
#pragma unroll
            for (int nt = 0; nt < 8; ++nt)
#pragma unroll
                for (int e = 0; e < 2; ++e) { sl += fast_exp2(s[nt][e] - nm_lo); sh += fast_exp2(s[nt][2 + e] - nm_hi); }
            l_lo = l_lo * fast_exp2(m_lo - nm_lo) + sl;
            l_hi = l_hi * fast_exp2(m_hi - nm_hi) + sh;
            m_lo = nm_lo; m_hi = nm_hi;
            __syncthreads();
        }
        l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1); l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
        l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1); l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
        const float lse_lo = m_lo + log2f(l_lo), lse_hi = m_hi + log2f(l_hi);

        // ---- pass 2: logp, KL, stored rows, P V ----------------------------------------------------------
        const bool with_v = a.out != nullptr;
        const bool vec = (a.N & 1) == 0;
        load_tile(0, with_v);
        if (n_tiles > 1) load_tile(1, with_v);
        if (n_tiles > 2) load_tile(2, with_v);
        for (int t = 0; t < n_tiles; ++t) {
            ring_step(t, with_v);
            float s[8][4];
            scores(t, s);
            uint32_t pf[4][4];
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {            // two halves of 4 key groups keep the register count down
                float pv_lo[4][2], pv_hi[4][2], lp_lo[4][2], lp_hi[4][2];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int key = t * BG_BN + (hf * 4 + u) * 8 + cpair;
                    pv_lo[u][0] = pv_lo[u][1] = pv_hi[u][0] = pv_hi[u][1] = 0.f;
                    if (a.record_kl) {
                        if (vec) {        // even N: the two keys of a thread are one 8-byte access
                            if (prev_lo && key < a.N) { const float2 v = *reinterpret_cast<const float2*>(prev_lo + key); pv_lo[u][0] = v.x; pv_lo[u][1] = v.y; }
                            if (prev_hi && key < a.N) { const float2 v = *reinterpret_cast<const float2*>(prev_hi + key); pv_hi[u][0] = v.x; pv_hi[u][1] = v.y; }
                        } else {
#pragma unroll
                            for (int e = 0; e < 2; ++e) {
                                if (prev_lo && key + e < a.N) pv_lo[u][e] = prev_lo[key + e];
                                if (prev_hi && key + e < a.N) pv_hi[u][e] = prev_hi[key + e];
                            }
                        }
                    }
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int nt = hf * 4 + u;
                    float p[4];
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const bool ok = t * BG_BN + nt * 8 + cpair + e < a.N;
                        const float d_lo = s[nt][e] * scale2 - lse_lo, d_hi = s[nt][2 + e] * scale2 - lse_hi;
                        const float p_lo = ok ? fast_exp2(d_lo) : 0.f, p_hi = ok ? fast_exp2(d_hi) : 0.f;
                        lp_lo[u][e] = d_lo * LN2; lp_hi[u][e] = d_hi * LN2;
                        if (ok && a.record_kl) {
                            if (prev_lo) kl_lo += p_lo * (lp_lo[u][e] - pv_lo[u][e]);
                            if (prev_hi) kl_hi += p_hi * (lp_hi[u][e] - pv_hi[u][e]);
                        }
                        p[e] = p_lo; p[2 + e] = p_hi;
                    }
                    pf[nt >> 1][(nt & 1) * 2 + 0] = pack_bf16(p[0], p[1]);
                    pf[nt >> 1][(nt & 1) * 2 + 1] = pack_bf16(p[2], p[3]);
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int key = t * BG_BN + (hf * 4 + u) * 8 + cpair;
                    if (vec) {
                        if (prev_lo && key < a.N) *reinterpret_cast<float2*>(prev_lo + key) = make_float2(lp_lo[u][0], lp_lo[u][1]);
                        if (prev_hi && key < a.N) *reinterpret_cast<float2*>(prev_hi + key) = make_float2(lp_hi[u][0], lp_hi[u][1]);
                    } else {
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            if (prev_lo && key + e < a.N) prev_lo[key + e] = lp_lo[u][e];
                            if (prev_hi && key + e < a.N) prev_hi[key + e] = lp_hi[u][e];
                        }
                    }
                }
            }
            if (a.out) pv(t, pf, o);
            __syncthreads();
        }
    }
    kl_lo += __shfl_xor_sync(0xffffffffu, kl_lo, 1); kl_lo += __shfl_xor_sync(0xffffffffu, kl_lo, 2);
    kl_hi += __shfl_xor_sync(0xffffffffu, kl_hi, 1); kl_hi += __shfl_xor_sync(0xffffffffu, kl_hi, 2);
    const bool v_lo = valid_sh[r_lo] != 0, v_hi = valid_sh[r_hi] != 0;
    if (a.out) {
#pragma unroll
        for (int nt = 0; nt < 16; ++nt) {
            const int col = h * AT_DH + nt * 8 + cpair;
            if (v_lo) *reinterpret_cast<__nv_bfloat162*>((__nv_bfloat16*)a.out + (size_t)(row0 + r_lo) * dq + col) = __floats2bfloat162_rn(o[nt][0], o[nt][1]);
            if (v_hi) *reinterpret_cast<__nv_bfloat162*>((__nv_bfloat16*)a.out + (size_t)(row0 + r_hi) * dq + col) = __floats2bfloat162_rn(o[nt][2], o[nt][3]);
        }
    }
    if (a.kl && (lane & 3) == 0) {
        if (v_lo) a.kl[(size_t)(row0 + r_lo) * a.n_heads + h] = (prev_lo && a.record_kl) ? kl_lo : 0.f;
        if (v_hi) a.kl[(size_t)(row0 + r_hi) * a.n_heads + h] = (prev_hi && a.record_kl) ? kl_hi : 0.f;
    }
}

template <int NW, int TPW, int CL = 1>
constexpr int sp_smem_bytes() { return NW * 2 * SP_SLOT_BYTES + AT_BM * AT_DH * 2 + (CL > 1 ? AT_BM * AT_DH * 4 : 0) + 1024; }

template <int NW, int TPW, int CL = 1>
static cudaError_t launch_attention_sp(const AttnMmaArgs& g, dim3 grid, cudaStream_t st) {
    constexpr int smem = sp_smem_bytes<NW, TPW, CL>();
    if (CL > 1) {
        grid.x *= CL;
        return launch_k_cluster(attention_sp_kernel<NW, TPW, CL>, grid, dim3(NW * 32), smem, st, (unsigned)CL, g);
    }
    return launch_k(attention_sp_kernel<NW, TPW, CL>, grid, dim3(NW * 32), smem, st, g);
}

// Dynamic shared-memory limits of the kernels above; once per device, before their first launch there.
static cudaError_t attention_mma_set_attributes() {
    cudaError_t e;
#define PS_ATTR(kern, bytes) if ((e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes)) != cudaSuccess) return e
    PS_ATTR((attention_sp_kernel<8, 1, 2>), (sp_smem_bytes<8, 1, 2>()));
    PS_ATTR((attention_sp_kernel<8, 2, 2>), (sp_smem_bytes<8, 2, 2>()));
    PS_ATTR((attention_sp_kernel<8, 2, 1>), (sp_smem_bytes<8, 2, 1>()));
    PS_ATTR((attention_sp_kernel<4, 4, 1>), (sp_smem_bytes<4, 4, 1>()));
    PS_ATTR((attention_sp_kernel<8, 4, 1>), (sp_smem_bytes<8, 4, 1>()));
    PS_ATTR(attention_big_kernel, BG_SMEM);
    PS_ATTR(attention_mma_kernel, AT_SMEM);
#undef PS_ATTR
    return cudaSuccess;
}

// mode: 0 automatic, 1 two-pass, 2 <8,2>, 3 <4,4>, 4 <8,4>, 5 many-rows, 6 / 7 key split over two CTAs
static cudaError_t launch_attention_mma(const AttnArgs& a, cudaStream_t st, int sm_count, int mode) {
    AttnMmaArgs g;
    g.a = a;
    const int batch = a.batch > 0 ? a.batch : 1;
    g.rows_per_seq = a.rows_per_seq > 0 ? a.rows_per_seq : a.n_rows;
    g.tiles_per_seq = (g.rows_per_seq + AT_BM - 1) / AT_BM;
    dim3 grid(g.tiles_per_seq * batch, a.n_heads);
    const long long ctas = (long long)grid.x * grid.y;
    // many rows per head (entry forwards, long sequences): share each K/V tile among 64 rows
    const long long big_ctas = (long long)((g.rows_per_seq + BG_BM - 1) / BG_BM) * batch * a.n_heads;
    if (mode == 5 || (mode == 0 && (a.N > 8 * 4 * AT_BN || ctas >= 4LL * sm_count) && g.rows_per_seq >= 48 && big_ctas >= sm_count)) {
        AttnMmaArgs gb = g;
        gb.tiles_per_seq = (g.rows_per_seq + BG_BM - 1) / BG_BM;
        return launch_k(attention_big_kernel, dim3(gb.tiles_per_seq * batch, a.n_heads), dim3(BG_WARPS * 32), BG_SMEM, st, gb);
    }
    if (mode != 1) {
        // few rows: split the keys of every (row tile, head) over a cluster of two CTAs
        if ((mode == 6 || (mode == 0 && 2 * ctas <= sm_count)) && a.N <= 2 * 8 * AT_BN) return launch_attention_sp<8, 1, 2>(g, grid, st);
        if ((mode == 7 || (mode == 0 && 2 * ctas <= sm_count)) && a.N <= 2 * 8 * 2 * AT_BN) return launch_attention_sp<8, 2, 2>(g, grid, st);
        // (one CTA of <8,2> per SM: beyond one wave the smaller <4,4> CTAs, three per SM, finish sooner)
        if ((mode == 2 || (mode == 0 && ctas <= sm_count)) && a.N <= 8 * 2 * AT_BN) return launch_attention_sp<8, 2>(g, grid, st);
        if ((mode == 3 || mode == 0) && a.N <= 4 * 4 * AT_BN) return launch_attention_sp<4, 4>(g, grid, st);
        if ((mode == 4 || mode == 0) && a.N <= 8 * 4 * AT_BN) return launch_attention_sp<8, 4>(g, grid, st);
    }
    return launch_k(attention_mma_kernel, grid, dim3(AT_WARPS * 32), AT_SMEM, st, g);
}

}  // namespace ps
