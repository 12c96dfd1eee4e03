// Shared device-side definitions of the Polestar step kernels.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace ps {

// ---- element types ---------------------------------------------------------------
template <typename T> __device__ __forceinline__ float to_f(T v);
template <> __device__ __forceinline__ float to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// two adjacent elements (even index) in one store
template <typename T> __device__ __forceinline__ void store_pair(T* p, float a, float b);
template <> __device__ __forceinline__ void store_pair<float>(float* p, float a, float b) {
    *reinterpret_cast<float2*>(p) = make_float2(a, b);
}
template <> __device__ __forceinline__ void store_pair<__nv_bfloat16>(__nv_bfloat16* p, float a, float b) {
    *reinterpret_cast<__nv_bfloat162*>(p) = __floats2bfloat162_rn(a, b);
}

// value a GEMM operand of type T actually carries (identity for float)
template <typename T> __device__ __forceinline__ float round_to(float v) { return to_f<T>(from_f<T>(v)); }

// ---- programmatic dependent launch -------------------------------------------------------
// Kernels of a forward are launched back to back with programmatic stream serialization: a
// kernel may start while its predecessor drains, and calls pdl_wait() before it touches anything
// the predecessor produced (the instructions are no-ops for ordinary launches).
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// ---- thread-block clusters: barrier over all threads of the cluster, distributed shared memory ---------
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t dsmem_addr(uint32_t local_addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ float4 ld_dsmem_f4(uint32_t addr) {
    float4 v;
    asm volatile("ld.shared::cluster.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ float2 ld_dsmem_f2(uint32_t addr) {
    float2 v;
    asm volatile("ld.shared::cluster.v2.f32 {%0,%1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}

// ---- optional kernel timeline (POLESTAR_TRACE builds only) ----------------------------------
// In a library built with -DPOLESTAR_TRACE, block 0 of every kernel records (kernel id, nanosecond time) once
// its dependencies are resolved; consecutive stamps give each kernel's real cost inside the pipeline.  The
// default build compiles none of this.
#ifdef POLESTAR_TRACE
__device__ long long* g_trace_buf = nullptr;   // [0] = next slot, then pairs (id, time)
__device__ __forceinline__ void trace_stamp(int id, int thread = 0) {
    long long* t = g_trace_buf;
    if (t && blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0 && threadIdx.x == thread) {
        const unsigned long long slot = atomicAdd((unsigned long long*)t, 1ULL);
        if (slot < 4000) {
            long long now;
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
            t[1 + 2 * slot] = id; t[2 + 2 * slot] = now;
        }
    }
}
#else
__device__ __forceinline__ void trace_stamp(int, int = 0) {}
#endif
#define KERNEL_PROLOGUE(id) do { pdl_trigger(); pdl_wait(); trace_stamp(id); } while (0)

// ---- rows of one forward -----------------------------------------------------------
// One descriptor per forwarded row.  pos < 0 marks an unused slot.
struct Row {
    int seq;   // sequence in the batch
    int pos;   // absolute position in the sequence, -1 = unused
    int widx;  // index in the local window, -1 = not a window row; <= -2: proxy row of cluster -2 - widx
    int aidx;  // index in the active block, -1 = not an active row
};
// Proxy rows (centroid proxies, Sec. 4.1 "Cluster and Quantize Hidden States") follow the ordinary rows of a
// sequence.  Their rotary position and emptiness differ from layer to layer (the clustering is per layer), so the
// row table only marks them; kernels look both up in the layer's cluster tables.
__device__ __forceinline__ bool row_is_proxy(int widx) { return widx <= -2; }
__device__ __forceinline__ int row_cluster(int widx) { return -2 - widx; }

struct SeqFlags { unsigned char v[64]; };

// Geometry of one forward (Algorithm 1: active block J_b, window Omega_b, entry set E_b).
struct StepDesc {
    int kind;          // 0 entry over the whole sequence, 1 entry over window+block, 2 within-block
    int batch, N, B;
    int act_start;     // first position of the active block
    int W, n_pre;      // window rows, of which the first n_pre lie before the block
    int pre_start;     // first position of the prefix part
    int suf_start;     // first position of the suffix part
    int W_max;         // row stride of the per-window buffers
    int rows_per_seq;  // descriptors per sequence
    int e0;            // entry steps: first forwarded position
    int within;        // 1: window rows live in the hidden cache (within-block step)
    int record_kl;     // 1: drift of recorded rows is measured against the stored rows
    int K;             // centroid proxies per sequence appended to the rows (0: per-position drift)
    SeqFlags refresh;  // within-block: which sequences refresh their cache this step
};

__device__ __forceinline__ int window_pos(const StepDesc& sd, int w) {
    return w < sd.n_pre ? sd.pre_start + w : sd.suf_start + (w - sd.n_pre);
}
__device__ __forceinline__ int window_index(const StepDesc& sd, int pos) {
    if (pos >= sd.pre_start && pos < sd.pre_start + sd.n_pre) return pos - sd.pre_start;
    if (pos >= sd.suf_start && pos < sd.suf_start + (sd.W - sd.n_pre)) return sd.n_pre + pos - sd.suf_start;
    return -1;
}

// ---- reductions (fixed order => deterministic) --------------------------------------
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
// sum over the whole block; every thread gets the result.  red: >= 33 floats of shared memory.
__device__ __forceinline__ float block_sum(float v, float* red) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
    v = warp_sum(v);
    __syncthreads();
    if (lane == 0) red[wid] = v;
    __syncthreads();
    if (wid == 0) {
        float t = lane < nw ? red[lane] : 0.f;
        t = warp_sum(t);
        if (lane == 0) red[32] = t;
    }
    __syncthreads();
    return red[32];
}
__device__ __forceinline__ float block_max(float v, float* red) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
    v = warp_max(v);
    __syncthreads();
    if (lane == 0) red[wid] = v;
    __syncthreads();
    if (wid == 0) {
        float t = lane < nw ? red[lane] : -INFINITY;
        t = warp_max(t);
        if (lane == 0) red[32] = t;
    }
    __syncthreads();
    return red[32];
}

// exclusive prefix sum of one int per thread over the block; returns the exclusive value,
// *total gets the block total.  sc: >= 33 ints of shared memory.
__device__ __forceinline__ int block_excl_scan(int v, int* sc, int* total) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
    int inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
    }
    __syncthreads();
    if (lane == 31) sc[wid] = inc;
    __syncthreads();
    if (wid == 0) {
        int t = lane < nw ? sc[lane] : 0;
        int ti = t;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int u = __shfl_up_sync(0xffffffffu, ti, o);
            if (lane >= o) ti += u;
        }
        if (lane < nw) sc[lane] = ti - t;
        if (lane == 31) sc[32] = ti;
    }
    __syncthreads();
    int res = inc - v + sc[wid];
    *total = sc[32];
    __syncthreads();
    return res;
}

// ---- GEMM epilogues -------------------------------------------------------------------
enum { EPI_QKV = 0, EPI_RESID = 1, EPI_SWIGLU = 2, EPI_DOWN = 3, EPI_LOGITS = 4, EPI_QKV_REFRESH = 5 };

// Everything an epilogue may need; unused members are null.
struct EpiArgs {
    const Row* rows;          // descriptors of the GEMM's rows (QKV) / of the forward (DOWN)
    const int* list;          // DOWN: compacted row -> forward row
    const int* m_count;       // device-side row count (null: use the host bound)
    const unsigned char* kvflag;  // QKV: write k,v of this row into the cache
    const float2* rope;       // [N][head_dim/2] (cos, sin)
    void* q_out;              // QKV: [rows][n_heads*head_dim]
    void* kc; void* vc;       // cache of this layer [batch][N][n_kv*head_dim]
    const float* resid;       // RESID / DOWN: residual rows [rows][d]
    float* out_f32;           // RESID: out rows; DOWN: x rows; LOGITS: logits
    float* packet;            // DOWN: packet rows [batch][W_max][d]
    void* out_t;              // SWIGLU: [rows][d_ffn]
    int N_seq, n_heads, n_kv, head_dim, W_max, within;
    int ld_out;               // leading dimension of the main output
    float scale;              // LOGITS
    // QKV_REFRESH (stand-alone refresh kernel): row r of sequence s = r / max_rows
    const int* idx; const int* counts; int max_rows; int P;
    // QKV with proxy rows: rotary position of cluster c of sequence s at zpos[s * n_clusters + c] (< 0: empty cluster)
    const int* zpos; int n_clusters;
    // RMSNorm folded into two GEMMs (steps whose rows all come straight from the previous GEMM): the producing
    // epilogue (RESID / DOWN) also stores a = x * gain in the model dtype and adds the row's sum of squares to
    // fold_ss (64-bit fixed point, 2^16: integer additions commute, so the sum is reproducible); the consuming
    // epilogue (SWIGLU / QKV) multiplies its rows by rsqrt(ss / d + eps), which commutes with the matrix product.
    void* fold_a; const float* fold_gain; long long* fold_ss;
    const long long* in_ss; float in_eps; int in_d;
    // RESID / DOWN whose output rows ARE the residual rows (out_f32 == resid, no packet rows in the step): every CTA
    // adds its part of the product straight onto them with vector reductions in L2 (red.global.add.v4.f32) -- no
    // published partial tiles, no wait for the other contributors, no reduction pass.  The order of the fp32
    // additions is then the order of arrival (results agree to rounding, not bit for bit).
    int accumulate;
};

constexpr float FOLD_SCALE = 65536.f;
// Adds `partial` (sum of squares of some columns of row `row`) to ss[row].  The lanes of the warp that hold the same
// row are added up first, in lane order, and one lane issues the integer atomic.
__device__ __forceinline__ void fold_ss_add(long long* ss, int row, float partial) {
    const unsigned act = __activemask();
    const unsigned grp = __match_any_sync(act, row);
    float sum = 0.f;
    for (unsigned rest = grp; rest; rest &= rest - 1) sum += __shfl_sync(grp, partial, __ffs(rest) - 1);
    if ((int)(threadIdx.x & 31) == __ffs(grp) - 1)
        atomicAdd(reinterpret_cast<unsigned long long*>(ss + row), (unsigned long long)__float2ll_rn(sum * FOLD_SCALE));
}
__device__ __forceinline__ float fold_inv(const EpiArgs& e, int m) {
    // (final before the consuming GEMM's first load; read through L1 so that epilogue_prefetch can have it waiting)
    const float ss = (float)e.in_ss[m] * (1.f / FOLD_SCALE);
    return rsqrtf(ss / (float)e.in_d + e.in_eps);
}

// Cluster tables of ONE layer (centroid proxies; all null / 0 in the per-position mode).
struct ClusterTabs {
    const int* labels;     // [batch][W_max] cluster of every window row
    const int* zpos;       // [batch][K] rotary position of the proxy (rounded mean of the members' positions), -1 = empty
    const int* zcnt;       // [batch][K] members
    const int* members;    // [batch][W_max] window indices grouped by cluster, ascending inside a cluster
    const int* moff;       // [batch][K + 1] start of every cluster's group
    float* zbuf;           // [batch][K][d] the proxy rows (member means), rebuilt whenever they are needed
    int K;
    // NVFP4 residual cache (null: the hidden cache holds plain fp32 rows): codes [batch][W_max][d/2] (two E2M1 values
    // per byte, low nibble first), E4M3 scale bytes [batch][W_max][d/16], reference rows [batch][K][d] = the
    // block-entry centroids
    unsigned char* hq; unsigned char* hs; float* z0;
    // imposed codes (null: none kept): rows whose mask byte is set take fq / fs (laid out like hq / hs) when encoded
    const unsigned char* fmask; const unsigned char* fq; const unsigned char* fs;
};

// ---- NVFP4 residual codec (Sec. 4.1 "Cluster and Quantize Hidden States"; Appendix "Quantization Format") ----
// E2M1 values {0, .5, 1, 1.5, 2, 3, 4, 6} with one FP8 E4M3 scale per 16 channels; float32 arithmetic throughout
// (the codes are integers decided by it): scale = E4M3(amax / 6), round to nearest even, saturating at 448; codes
// round to the nearest grid value, ties to the even code, saturating at 6.
__device__ __forceinline__ float e4m3_round_pos(float x) {          // x >= 0 -> nearest E4M3 value
    x = fminf(x, 448.f);
    if (x < 0.015625f) return rintf(x * 512.f) * 0.001953125f;       // below 2^-6: multiples of 2^-9 (both products exact)
    // normal range: keep 3 mantissa bits, round to nearest even (a carry moves on to the exponent)
    unsigned b = __float_as_uint(x);
    b += 0x7FFFFu + ((b >> 20) & 1u);
    return fminf(__uint_as_float(b & 0xFFF00000u), 448.f);
}
__device__ __forceinline__ unsigned e4m3_bits(float q) {            // q on the E4M3 grid, >= 0
    if (q < 0.015625f) return (unsigned)(q * 512.f);                 // subnormal: m 2^-9
    const unsigned b = __float_as_uint(q);
    return (((b >> 23) - 120u) << 3) | ((b >> 20) & 7u);             // exponent bias 127 -> 7
}
__device__ __forceinline__ float e4m3_value(unsigned b) {
    const unsigned e = (b >> 3) & 15u, m = b & 7u;
    return e == 0 ? (float)m * 0.001953125f : __uint_as_float(((e + 120u) << 23) | (m << 20));
}
__device__ __forceinline__ unsigned e2m1_code(float r, float s) {   // residual r, group scale s > 0 -> sign | index
    const float y = __fdiv_rn(fabsf(r), s);
    unsigned i = (y > 0.25f) + (y >= 0.75f) + (y > 1.25f) + (y >= 1.75f) + (y > 2.5f) + (y >= 3.5f) + (y > 5.f);
    return i | (r < 0.f ? 8u : 0u);
}
__device__ __forceinline__ float e2m1_value(unsigned code, float s) {
    // index = 2 bits of exponent, 1 of mantissa: 0, .5 | (1 + m / 2) 2^(e - 1)
    const unsigned e = (code >> 1) & 3u, m = code & 1u;
    const float g = e == 0 ? 0.5f * (float)m : __uint_as_float(((e + 126u) << 23) | (m << 22));
    return __uint_as_float(__float_as_uint(g * s) | ((code & 8u) << 28));
}
// One 16-byte chunk (4 channels) of a row; the 4 lanes that hold a group of 16 channels call together (lane % 4 =
// position in the group; every lane of the warp takes part).  Returns the stored value ref + dequant(quant(v - ref));
// *codes = the chunk's four codes (4 bits each, channel 0 lowest), *scale_bits = the group's E4M3 byte.
__device__ __forceinline__ float4 nvfp4_residual_chunk(float4 v, float4 ref, unsigned* codes, unsigned* scale_bits) {
    const float4 r = make_float4(v.x - ref.x, v.y - ref.y, v.z - ref.z, v.w - ref.w);
    float am = fmaxf(fmaxf(fabsf(r.x), fabsf(r.y)), fmaxf(fabsf(r.z), fabsf(r.w)));
    am = fmaxf(am, __shfl_xor_sync(0xffffffffu, am, 1));
    am = fmaxf(am, __shfl_xor_sync(0xffffffffu, am, 2));
    const float s = e4m3_round_pos(__fdiv_rn(am, 6.f));
    *scale_bits = e4m3_bits(s);
    if (!(s > 0.f)) { *codes = 0u; return ref; }
    const unsigned c0 = e2m1_code(r.x, s), c1 = e2m1_code(r.y, s), c2 = e2m1_code(r.z, s), c3 = e2m1_code(r.w, s);
    *codes = c0 | (c1 << 4) | (c2 << 8) | (c3 << 12);
    return make_float4(ref.x + e2m1_value(c0, s), ref.y + e2m1_value(c1, s), ref.z + e2m1_value(c2, s), ref.w + e2m1_value(c3, s));
}
__device__ __forceinline__ float4 nvfp4_dequant_chunk(unsigned codes, unsigned scale_bits, float4 ref) {
    const float s = e4m3_value(scale_bits);
    return make_float4(ref.x + e2m1_value(codes & 15u, s), ref.y + e2m1_value((codes >> 4) & 15u, s),
                       ref.z + e2m1_value((codes >> 8) & 15u, s), ref.w + e2m1_value((codes >> 12) & 15u, s));
}

// Row-wise work appended to a GEMM whose output rows are the input of the next normalisation: once every CTA
// of the grid has stored its outputs (a counter all CTAs add to), the CTAs share out the rows and stage the
// next GEMM's operand, which saves a kernel boundary per normalisation.
//   kind 1: RMSNorm of the finished rows (FFN input);  kind 2: patch + RMSNorm + staging of the next layer's
//   QKV input (Algorithm 1 "Patch").  kind 0: nothing.
struct PostArgs {
    int kind, n_rows, d;
    float eps;
    const float* gain;
    void* a_out;
    float* x;                                  // rows written by this GEMM (kind 1: source; kind 2: residual stream)
    const int* list; const int* m_count;       // kind 1
    const Row* rows; float* hc; const float* packet; const unsigned char* patch; unsigned char* kvflag;   // kind 2
    StepDesc sd;                               // kind 2
    ClusterTabs ct;                            // kind 2: cluster tables of the layer being staged
    unsigned* counter;                         // never reset: `expect` is the running total after this launch
    unsigned expect;
};

// SwiGLU of one (gate, up) pair: silu(g) * u with the hardware exponential and reciprocal (relative error ~1e-6, far below
// the rounding of the stored result); the full-precision expf and division made the gate/up epilogue instruction-bound.
__device__ __forceinline__ float swiglu(float g, float u) { return __fdividef(g, 1.f + __expf(-g)) * u; }

// One output pair (n even, n+1) of row m.
template <typename T, int EPI>
__device__ __forceinline__ void epilogue_pair(const EpiArgs& e, int m, int n, float v0, float v1) {
    if (EPI == EPI_QKV || EPI == EPI_QKV_REFRESH) {
        int seq, pos, kvf, qrow;
        if (EPI == EPI_QKV) {
            const int4 rw = __ldg(reinterpret_cast<const int4*>(e.rows) + m);   // {seq, pos, widx, aidx}
            if (rw.y < 0) return;
            seq = rw.x; pos = rw.y; kvf = __ldg(e.kvflag + m); qrow = m;
            if (row_is_proxy(rw.z)) { pos = __ldg(e.zpos + seq * e.n_clusters + row_cluster(rw.z)); kvf = 0; if (pos < 0) return; }
        } else {
            seq = m / e.max_rows;
            const int i = m - seq * e.max_rows;
            if (i >= __ldg(e.counts + seq)) return;
            pos = __ldg(e.idx + seq * e.max_rows + i); kvf = 1; qrow = m;
        }
        const int dq = e.n_heads * e.head_dim, dkv = e.n_kv * e.head_dim;
        const int Npos = (EPI == EPI_QKV) ? e.N_seq : e.P;
        if (n < dq + dkv) {
            const int hd1 = e.head_dim - 1;
            const int p = (e.head_dim & hd1) ? n % e.head_dim : (n & hd1);      // power-of-two head sizes: no division
            const float2 cs = __ldg(e.rope + (size_t)pos * (e.head_dim / 2) + (p >> 1));
            const float r0 = v0 * cs.x - v1 * cs.y;
            const float r1 = v1 * cs.x + v0 * cs.y;
            if (n < dq) {
                if (e.q_out) {
                    store_pair<T>((T*)e.q_out + (size_t)qrow * dq + n, r0, r1);
                }
            } else if (kvf) {
                store_pair<T>((T*)e.kc + ((size_t)seq * Npos + pos) * dkv + (n - dq), r0, r1);
            }
        } else if (kvf) {
            store_pair<T>((T*)e.vc + ((size_t)seq * Npos + pos) * dkv + (n - dq - dkv), v0, v1);
        }
    } else if (EPI == EPI_RESID) {
        const size_t o = (size_t)m * e.ld_out + n;
        const float2 r = __ldg(reinterpret_cast<const float2*>(e.resid + o));
        *reinterpret_cast<float2*>(e.out_f32 + o) = make_float2(r.x + v0, r.y + v1);
    } else if (EPI == EPI_SWIGLU) {
        const float g = swiglu(v0, v1);
        ((T*)e.out_t)[(size_t)m * e.ld_out + (n >> 1)] = from_f<T>(g);
    } else if (EPI == EPI_DOWN) {
        const int r = e.list ? __ldg(e.list + m) : m;
        const int4 rw = __ldg(reinterpret_cast<const int4*>(e.rows) + r);       // {seq, pos, widx, aidx}
        if (rw.y < 0) return;
        const size_t o = (size_t)r * e.ld_out + n;
        const float2 rs = __ldg(reinterpret_cast<const float2*>(e.resid + o));
        float* dst = (e.within && rw.z >= 0)
                         ? e.packet + ((size_t)rw.x * e.W_max + rw.z) * e.ld_out + n
                         : e.out_f32 + o;
        *reinterpret_cast<float2*>(dst) = make_float2(rs.x + v0, rs.y + v1);
    } else if (EPI == EPI_LOGITS) {
        const size_t o = (size_t)m * e.ld_out + n;
        *reinterpret_cast<float2*>(e.out_f32 + o) = make_float2(v0 * e.scale, v1 * e.scale);
    }
}

// 16 consecutive values to dst (16-byte aligned)
template <typename T> __device__ __forceinline__ void store16(T* dst, const float* v);
template <> __device__ __forceinline__ void store16<float>(float* dst, const float* v) {
#pragma unroll
    for (int i = 0; i < 4; ++i) reinterpret_cast<float4*>(dst)[i] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
}
template <> __device__ __forceinline__ void store16<__nv_bfloat16>(__nv_bfloat16* dst, const float* v) {
    uint32_t w[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        __nv_bfloat162 b = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
        w[i] = *reinterpret_cast<uint32_t*>(&b);
    }
    reinterpret_cast<uint4*>(dst)[0] = make_uint4(w[0], w[1], w[2], w[3]);
    reinterpret_cast<uint4*>(dst)[1] = make_uint4(w[4], w[5], w[6], w[7]);
}
template <typename T> __device__ __forceinline__ void store8(T* dst, const float* v);
template <> __device__ __forceinline__ void store8<float>(float* dst, const float* v) {
    reinterpret_cast<float4*>(dst)[0] = make_float4(v[0], v[1], v[2], v[3]);
    reinterpret_cast<float4*>(dst)[1] = make_float4(v[4], v[5], v[6], v[7]);
}
template <> __device__ __forceinline__ void store8<__nv_bfloat16>(__nv_bfloat16* dst, const float* v) {
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        __nv_bfloat162 b = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
        w[i] = *reinterpret_cast<uint32_t*>(&b);
    }
    reinterpret_cast<uint4*>(dst)[0] = make_uint4(w[0], w[1], w[2], w[3]);
}

// producing side of the folded RMSNorm: a = x * gain for 16 (4) finished values of row `row`, and their squares
template <typename T>
__device__ __forceinline__ void fold_store16(const EpiArgs& e, int row, size_t o, int n, const float* r) {
    float a16[16];
    float ss = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float4 g = __ldg(reinterpret_cast<const float4*>(e.fold_gain + n) + i);
        a16[4 * i] = r[4 * i] * g.x; a16[4 * i + 1] = r[4 * i + 1] * g.y; a16[4 * i + 2] = r[4 * i + 2] * g.z; a16[4 * i + 3] = r[4 * i + 3] * g.w;
        ss += r[4 * i] * r[4 * i] + r[4 * i + 1] * r[4 * i + 1] + r[4 * i + 2] * r[4 * i + 2] + r[4 * i + 3] * r[4 * i + 3];
    }
    store16<T>((T*)e.fold_a + o, a16);
    fold_ss_add(e.fold_ss, row, ss);
}
template <typename T>
__device__ __forceinline__ void fold_store4(const EpiArgs& e, int row, size_t o, int n, float4 r) {
    const float4 g = __ldg(reinterpret_cast<const float4*>(e.fold_gain + n));
    T* dst = (T*)e.fold_a + o;
    store_pair<T>(dst, r.x * g.x, r.y * g.y);
    store_pair<T>(dst + 2, r.z * g.z, r.w * g.w);
    fold_ss_add(e.fold_ss, row, r.x * r.x + r.y * r.y + r.z * r.z + r.w * r.w);
}

// The 16 outputs n .. n+15 (n % 16 == 0) of row m: the same arithmetic as epilogue_pair on each pair, with the
// row descriptor read once and all loads and stores 16 bytes wide.  Requires head_dim % 16 == 0 and leading
// dimensions that keep 16-column groups 16-byte aligned (true for every matrix the tensor-core path accepts).
template <typename T, int EPI>
__device__ __forceinline__ void epilogue16(const EpiArgs& e, int m, int n, const float* v) {
    if (EPI == EPI_QKV || EPI == EPI_QKV_REFRESH) {
        int seq, pos, kvf;
        if (EPI == EPI_QKV) {
            const int4 rw = __ldg(reinterpret_cast<const int4*>(e.rows) + m);   // {seq, pos, widx, aidx}
            if (rw.y < 0) return;
            seq = rw.x; pos = rw.y; kvf = __ldg(e.kvflag + m);
            if (row_is_proxy(rw.z)) { pos = __ldg(e.zpos + seq * e.n_clusters + row_cluster(rw.z)); kvf = 0; if (pos < 0) return; }
        } else {
            seq = m / e.max_rows;
            const int i = m - seq * e.max_rows;
            if (i >= __ldg(e.counts + seq)) return;
            pos = __ldg(e.idx + seq * e.max_rows + i); kvf = 1;
        }
        const int dq = e.n_heads * e.head_dim, dkv = e.n_kv * e.head_dim;
        const int Npos = (EPI == EPI_QKV) ? e.N_seq : e.P;
        float vs[16];
        {
            const float inv = (EPI == EPI_QKV && e.in_ss) ? fold_inv(e, m) : 1.f;
#pragma unroll
            for (int i = 0; i < 16; ++i) vs[i] = v[i] * inv;
        }
        v = vs;
        if (n < dq + dkv) {
            if (n < dq ? e.q_out == nullptr : !kvf) return;
            const int hd1 = e.head_dim - 1;
            const int p = (e.head_dim & hd1) ? n % e.head_dim : (n & hd1);
            const float4* cs = reinterpret_cast<const float4*>(e.rope + (size_t)pos * (e.head_dim / 2) + (p >> 1));
            float r[16];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float4 c = __ldg(cs + i);          // (cos, sin) of two pairs
                r[4 * i] = v[4 * i] * c.x - v[4 * i + 1] * c.y;
                r[4 * i + 1] = v[4 * i + 1] * c.x + v[4 * i] * c.y;
                r[4 * i + 2] = v[4 * i + 2] * c.z - v[4 * i + 3] * c.w;
                r[4 * i + 3] = v[4 * i + 3] * c.z + v[4 * i + 2] * c.w;
            }
            if (n < dq) store16<T>((T*)e.q_out + (size_t)m * dq + n, r);
            else store16<T>((T*)e.kc + ((size_t)seq * Npos + pos) * dkv + (n - dq), r);
        } else if (kvf) {
            store16<T>((T*)e.vc + ((size_t)seq * Npos + pos) * dkv + (n - dq - dkv), v);
        }
    } else if (EPI == EPI_RESID) {
        const size_t o = (size_t)m * e.ld_out + n;
        float r[16];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float4 c = __ldg(reinterpret_cast<const float4*>(e.resid + o) + i);
            r[4 * i] = c.x + v[4 * i]; r[4 * i + 1] = c.y + v[4 * i + 1]; r[4 * i + 2] = c.z + v[4 * i + 2]; r[4 * i + 3] = c.w + v[4 * i + 3];
        }
        store16<float>(e.out_f32 + o, r);
        if (e.fold_a) fold_store16<T>(e, m, o, n, r);
    } else if (EPI == EPI_SWIGLU) {
        const float inv = e.in_ss ? fold_inv(e, m) : 1.f;
        float gl[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float ga = v[2 * i] * inv, up = v[2 * i + 1] * inv;
            gl[i] = swiglu(ga, up);
        }
        store8<T>((T*)e.out_t + (size_t)m * e.ld_out + (n >> 1), gl);
    } else if (EPI == EPI_DOWN) {
        const int r0 = e.list ? __ldg(e.list + m) : m;
        const int4 rw = __ldg(reinterpret_cast<const int4*>(e.rows) + r0);       // {seq, pos, widx, aidx}
        if (rw.y < 0) return;
        const size_t o = (size_t)r0 * e.ld_out + n;
        float r[16];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float4 c = __ldg(reinterpret_cast<const float4*>(e.resid + o) + i);
            r[4 * i] = c.x + v[4 * i]; r[4 * i + 1] = c.y + v[4 * i + 1]; r[4 * i + 2] = c.z + v[4 * i + 2]; r[4 * i + 3] = c.w + v[4 * i + 3];
        }
        float* dst = (e.within && rw.z >= 0) ? e.packet + ((size_t)rw.x * e.W_max + rw.z) * e.ld_out + n : e.out_f32 + o;
        store16<float>(dst, r);
        if (e.fold_a && !(e.within && rw.z >= 0)) fold_store16<T>(e, r0, o, n, r);
    } else if (EPI == EPI_LOGITS) {
        float r[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) r[i] = v[i] * e.scale;
        store16<float>(e.out_f32 + (size_t)m * e.ld_out + n, r);
    }
}

// Four outputs n .. n+3 (n % 4 == 0) of row m for the two residual epilogues (same arithmetic as epilogue16).
template <typename T, int EPI>
__device__ __forceinline__ void epilogue4(const EpiArgs& e, int m, int n, float4 v) {
    if (EPI == EPI_RESID) {
        const size_t o = (size_t)m * e.ld_out + n;
        const float4 c = __ldg(reinterpret_cast<const float4*>(e.resid + o));
        const float4 r = make_float4(c.x + v.x, c.y + v.y, c.z + v.z, c.w + v.w);
        *reinterpret_cast<float4*>(e.out_f32 + o) = r;
        if (e.fold_a) fold_store4<T>(e, m, o, n, r);
    } else if (EPI == EPI_DOWN) {
        const int r0 = e.list ? __ldg(e.list + m) : m;
        const int4 rw = __ldg(reinterpret_cast<const int4*>(e.rows) + r0);       // {seq, pos, widx, aidx}
        if (rw.y < 0) return;
        const size_t o = (size_t)r0 * e.ld_out + n;
        const float4 c = __ldg(reinterpret_cast<const float4*>(e.resid + o));
        float* dst = (e.within && rw.z >= 0) ? e.packet + ((size_t)rw.x * e.W_max + rw.z) * e.ld_out + n : e.out_f32 + o;
        const float4 r = make_float4(c.x + v.x, c.y + v.y, c.z + v.z, c.w + v.w);
        *reinterpret_cast<float4*>(dst) = r;
        if (e.fold_a && !(e.within && rw.z >= 0)) fold_store4<T>(e, r0, o, n, r);
    }
}

// Prefetch into L1 what epilogue_pair will read for the 16 outputs n .. n+15 of row m (row descriptor,
// RoPE entries, residual values), so that the epilogue after a wait starts on cache hits.
__device__ __forceinline__ void prefetch_l1(const void* p) { asm volatile("prefetch.global.L1 [%0];" ::"l"(p)); }
template <typename T, int EPI>
__device__ __forceinline__ void epilogue_prefetch(const EpiArgs& e, int m, int n) {
    if (EPI == EPI_QKV) {
        const int4 rw = __ldg(reinterpret_cast<const int4*>(e.rows) + m);
        prefetch_l1(e.kvflag + m);
        if (e.in_ss) prefetch_l1(e.in_ss + m);
        if (rw.y >= 0 && n < (e.n_heads + e.n_kv) * e.head_dim)
            prefetch_l1(e.rope + (size_t)rw.y * (e.head_dim / 2) + ((n % e.head_dim) >> 1));
    } else if (EPI == EPI_RESID) {
        prefetch_l1(e.resid + (size_t)m * e.ld_out + n);
        if (e.fold_a) prefetch_l1(e.fold_gain + n);
    } else if (EPI == EPI_DOWN) {
        const int r = e.list ? __ldg(e.list + m) : m;
        prefetch_l1(reinterpret_cast<const int4*>(e.rows) + r);
        prefetch_l1(e.resid + (size_t)r * e.ld_out + n);
        if (e.fold_a) prefetch_l1(e.fold_gain + n);
    } else if (EPI == EPI_SWIGLU) {
        if (e.in_ss) prefetch_l1(e.in_ss + m);
    }
}

// ---- host: launch with programmatic stream serialization -----------------------------------
inline bool g_use_pdl = true;
template <typename... KArgs, typename... Args>
static cudaError_t launch_k(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = g_use_pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}
// same, with the grid grouped into thread-block clusters of `cluster` consecutive CTAs
template <typename... KArgs, typename... Args>
static cudaError_t launch_k_cluster(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                    unsigned cluster, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute at[2];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = cluster; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = g_use_pdl ? 2 : 1;
    return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

}  // namespace ps
