// CUDA-core kernels of the Polestar step: row table, embedding, RMSNorm staging, a plain
// tiled GEMM (fp32 models and debugging), attention with drift (fp32 models), select /
// compaction, confidence and commit.
#pragma once
#include "common.cuh"

namespace ps {

// ---------------------------------------------------------------------------------------
// Row table of one forward (Algorithm 1: E_b at block entry, J_b plus Omega_b within a block)
// ---------------------------------------------------------------------------------------
__global__ void build_rows_kernel(StepDesc sd, Row* rows) {
    KERNEL_PROLOGUE(1);   // build_rows_kernel
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    const int total = sd.batch * sd.rows_per_seq;
    if (i >= total) return;
    const int s = i / sd.rows_per_seq, j = i - s * sd.rows_per_seq;
    Row r;
    r.seq = s; r.pos = -1; r.widx = -1; r.aidx = -1;
    const int n_plain = sd.rows_per_seq - sd.K;      // the proxy rows of the clusters come last
    if (j >= n_plain) {
        // proxy row: position and emptiness are per layer (cluster tables); unused on steps without refresh
        if (sd.kind != 2 || sd.refresh.v[s]) { r.pos = 0; r.widx = -2 - (j - n_plain); }
    } else if (sd.kind == 2) {
        if (j < sd.B) {
            r.pos = sd.act_start + j; r.aidx = j;
        } else {
            const int w = j - sd.B;
            if (w < sd.W && sd.refresh.v[s]) { r.pos = window_pos(sd, w); r.widx = w; }
        }
    } else {
        const int pos = sd.e0 + j;
        if (pos < sd.N) {
            r.pos = pos;
            if (pos >= sd.act_start && pos < sd.act_start + sd.B) r.aidx = pos - sd.act_start;
            else r.widx = window_index(sd, pos);
        }
    }
    rows[i] = r;
}

// ---------------------------------------------------------------------------------------
// Layer-0 inputs: embeddings of forwarded rows; on refresh steps the layer-0 packet holds the
// embeddings of window positions whose token changed since their cached row was written
// ---------------------------------------------------------------------------------------
template <typename T>
__global__ void embed_rows_kernel(StepDesc sd, const Row* rows, const int* y, const T* emb, int d,
                                  float* x, float* packet, unsigned char* patch0, int* tok_at_h0,
                                  int* stats) {
    KERNEL_PROLOGUE(2);   // embed_rows_kernel
    const int r = blockIdx.x;
    const Row rw = rows[r];
    if (rw.pos < 0 || row_is_proxy(rw.widx)) return;
    const int tok = y[rw.seq * sd.N + rw.pos];
    const T* e = emb + (size_t)tok * d;
    if (sd.within && rw.widx >= 0) {
        const int o = rw.seq * sd.W_max + rw.widx;
        const bool changed = tok_at_h0[o] != tok;
        if (changed) {
            float* dst = packet + (size_t)o * d;
            for (int c = threadIdx.x; c < d; c += blockDim.x) dst[c] = to_f<T>(e[c]);
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            patch0[o] = changed ? 1 : 0;
            tok_at_h0[o] = tok;
            if (changed) atomicAdd(stats, 1);
        }
    } else {
        float* dst = x + (size_t)r * d;
        for (int c = threadIdx.x; c < d; c += blockDim.x) dst[c] = to_f<T>(e[c]);
        if (!sd.within && rw.widx >= 0 && threadIdx.x == 0) tok_at_h0[rw.seq * sd.W_max + rw.widx] = tok;
    }
}

// ---------------------------------------------------------------------------------------
// One row of RMSNorm + staging, held in registers: every thread owns up to NORM_VPT float4 chunks,
// so the row is read once (all loads in flight together), reduced, scaled and stored.
// Requires d % 4 == 0 and d <= 4 * NORM_VPT * blockDim.x.
// ---------------------------------------------------------------------------------------
constexpr int NORM_THREADS = 512;
constexpr int NORM_VPT = 8;
template <typename T>
__device__ __forceinline__ void store4(T* p, float a, float b, float c, float d4);
template <>
__device__ __forceinline__ void store4<float>(float* p, float a, float b, float c, float d4) {
    *reinterpret_cast<float4*>(p) = make_float4(a, b, c, d4);
}
template <>
__device__ __forceinline__ void store4<__nv_bfloat16>(__nv_bfloat16* p, float a, float b, float c, float d4) {
    __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c, d4);
    uint2 u;
    u.x = *reinterpret_cast<uint32_t*>(&lo);
    u.y = *reinterpret_cast<uint32_t*>(&hi);
    *reinterpret_cast<uint2*>(p) = u;
}
// src row -> a_out row (normed, times gain); optional copies of the raw row to up to two fp32 destinations
template <typename T>
__device__ __forceinline__ void norm_row(const float* __restrict__ src, const float* __restrict__ gain, float eps, int d,
                                         T* a_out, float* copy0, float* copy1, float* red) {
    const int n4 = d >> 2;
    float4 v[NORM_VPT];
    float ss = 0.f;
#pragma unroll
    for (int u = 0; u < NORM_VPT; ++u) {
        const int c4 = threadIdx.x + u * blockDim.x;
        v[u] = c4 < n4 ? __ldcg(reinterpret_cast<const float4*>(src) + c4) : make_float4(0.f, 0.f, 0.f, 0.f);
        // the gains are needed only after the reduction: have them in L1 by then
        if (c4 < n4) asm volatile("prefetch.global.L1 [%0];" ::"l"(reinterpret_cast<const float4*>(gain) + c4));
    }
#pragma unroll
    for (int u = 0; u < NORM_VPT; ++u) ss += v[u].x * v[u].x + v[u].y * v[u].y + v[u].z * v[u].z + v[u].w * v[u].w;
    ss = block_sum(ss, red);
    const float inv = rsqrtf(ss / (float)d + eps);
#pragma unroll
    for (int u = 0; u < NORM_VPT; ++u) {
        const int c4 = threadIdx.x + u * blockDim.x;
        if (c4 < n4) {
            const float4 g = __ldg(reinterpret_cast<const float4*>(gain) + c4);
            store4<T>(a_out + 4 * c4, v[u].x * inv * g.x, v[u].y * inv * g.y, v[u].z * inv * g.z, v[u].w * inv * g.w);
            if (copy0) reinterpret_cast<float4*>(copy0)[c4] = v[u];
            if (copy1) reinterpret_cast<float4*>(copy1)[c4] = v[u];
        }
    }
}
template <typename T>
__device__ __forceinline__ void zero_row(T* a, int d) {
    for (int c = threadIdx.x; c < d; c += blockDim.x) a[c] = from_f<T>(0.f);
}

// ---------------------------------------------------------------------------------------
// Patch + RMSNorm + staging of the QKV projection's input rows (Algorithm 1 "Patch")
//   window rows of a within-block step read the hidden cache (after taking the packet row if
//   the previous layer selected them); every other row reads the residual stream x.
// ---------------------------------------------------------------------------------------
template <typename T>
__device__ __forceinline__ void prep_qkv_row(const StepDesc& sd, int r, const Row* rows, float* x, float* hc, const float* packet,
                                             const unsigned char* patch, const float* gain, float eps, int d,
                                             T* a_out, unsigned char* kvflag, float* red, const ClusterTabs& ct) {
    const Row rw = rows[r];
    T* a = a_out + (size_t)r * d;
    if (rw.pos < 0) {
        zero_row<T>(a, d);
        if (threadIdx.x == 0) kvflag[r] = 0;
        return;
    }
    if (row_is_proxy(rw.widx)) {
        // Proxy of a cluster = mean of its members' current hidden rows (Sec. 4.1: the centroid follows its refreshed
        // members; rebuilding the mean from the cache is that incremental update without its rounding drift).
        // Members are added in ascending window order by every thread for its own columns: deterministic.
        const int c = row_cluster(rw.widx);
        const int n = ct.zcnt[rw.seq * ct.K + c];
        if (threadIdx.x == 0) kvflag[r] = 0;
        if (n <= 0) { zero_row<T>(a, d); return; }
        const int* mem = ct.members + (size_t)rw.seq * sd.W_max + ct.moff[rw.seq * (ct.K + 1) + c];
        float* z = ct.zbuf + ((size_t)rw.seq * ct.K + c) * d;
        const float inv_n = 1.f / (float)n;
        const int n4 = d >> 2;
        // the members' row tables go through shared memory in groups, so that the loads of the rows themselves do not
        // wait on a chain of dependent index loads
        constexpr int GROUP = 64;
        __shared__ const float* s_src[GROUP];
        __shared__ int s_o[GROUP];                               // row of the cache; bit 30: the row enters the cache now
        float4 acc[NORM_VPT], rf[NORM_VPT];
#pragma unroll
        for (int u = 0; u < NORM_VPT; ++u) {
            const int c4 = threadIdx.x + u * blockDim.x;
            acc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
            rf[u] = (ct.hq && c4 < n4) ? __ldg(reinterpret_cast<const float4*>(ct.z0 + ((size_t)rw.seq * ct.K + c) * d) + c4)
                                       : make_float4(0.f, 0.f, 0.f, 0.f);
        }
        for (int t0 = 0; t0 < n; t0 += GROUP) {
            __syncthreads();
            if (threadIdx.x < GROUP && t0 + threadIdx.x < n) {
                const int w = mem[t0 + threadIdx.x];
                const int o = rw.seq * sd.W_max + w;
                const bool pt = sd.within && patch[o];
                s_src[threadIdx.x] = !sd.within ? x + ((size_t)rw.seq * sd.rows_per_seq + (window_pos(sd, w) - sd.e0)) * d
                                                : (pt ? packet + (size_t)o * d : hc + (size_t)o * d);
                s_o[threadIdx.x] = o | ((!sd.within || pt) ? (1 << 30) : 0);
            }
            __syncthreads();
            const int nb = min(GROUP, n - t0);
#pragma unroll
            for (int u = 0; u < NORM_VPT; ++u) {
                const int c4 = threadIdx.x + u * blockDim.x;
                const bool in = c4 < n4;
                if (u * (int)blockDim.x >= n4) continue;         // (the whole block is past the row)
                // members in ascending window order for every column (deterministic), four at a time: all loads of a
                // group are issued before the first of them is used
                for (int t = 0; t < nb; t += 4) {
                    float4 v[4];
                    unsigned cd[4], sb[4];
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        v[k] = make_float4(0.f, 0.f, 0.f, 0.f);
                        cd[k] = sb[k] = 0;
                        if (t + k < nb && in) {
                            const int so = s_o[t + k];
                            const size_t o = (size_t)(so & ~(1 << 30));
                            const bool fresh = (so >> 30) & 1;
                            if (!ct.hq || fresh) v[k] = __ldcg(reinterpret_cast<const float4*>(s_src[t + k]) + c4);
                            if (ct.hq) {
                                // the member's STORED value: the codes in the cache, or (a row that enters the cache in this
                                // step) what the codec makes of the plain row, or the codes imposed on it
                                const bool imposed = fresh && ct.fmask && ct.fmask[o];
                                const unsigned char* q = imposed ? ct.fq : ct.hq;
                                const unsigned char* sc = imposed ? ct.fs : ct.hs;
                                if (!fresh || imposed) {
                                    cd[k] = *reinterpret_cast<const unsigned short*>(q + o * (size_t)(d >> 1) + 2 * c4);
                                    sb[k] = sc[o * (size_t)(d >> 4) + (c4 >> 2)];
                                }
                            }
                        }
                    }
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        if (t + k < nb) {                        // (uniform: the codec's lanes act together)
                            if (ct.hq) {
                                const int so = s_o[t + k];
                                const bool fresh = (so >> 30) & 1;
                                const bool imposed = fresh && ct.fmask && ct.fmask[(size_t)(so & ~(1 << 30))];
                                if (fresh && !imposed) {
                                    unsigned c_, s_;
                                    v[k] = nvfp4_residual_chunk(v[k], rf[u], &c_, &s_);
                                } else if (in) {
                                    v[k] = nvfp4_dequant_chunk(cd[k], sb[k], rf[u]);
                                }
                            }
                            acc[u].x += v[k].x; acc[u].y += v[k].y; acc[u].z += v[k].z; acc[u].w += v[k].w;
                        }
                    }
                }
            }
        }
        // the mean row (kept for read-back) and its RMSNorm, straight from the registers
        float ss = 0.f;
#pragma unroll
        for (int u = 0; u < NORM_VPT; ++u) {
            const int c4 = threadIdx.x + u * blockDim.x;
            acc[u] = make_float4(acc[u].x * inv_n, acc[u].y * inv_n, acc[u].z * inv_n, acc[u].w * inv_n);
            if (c4 < n4) {
                reinterpret_cast<float4*>(z)[c4] = acc[u];
                ss += acc[u].x * acc[u].x + acc[u].y * acc[u].y + acc[u].z * acc[u].z + acc[u].w * acc[u].w;
            }
        }
        ss = block_sum(ss, red);
        const float inv = rsqrtf(ss / (float)d + eps);
#pragma unroll
        for (int u = 0; u < NORM_VPT; ++u) {
            const int c4 = threadIdx.x + u * blockDim.x;
            if (c4 < n4) {
                const float4 g = __ldg(reinterpret_cast<const float4*>(gain) + c4);
                store4<T>(a + 4 * c4, acc[u].x * inv * g.x, acc[u].y * inv * g.y, acc[u].z * inv * g.z, acc[u].w * inv * g.w);
            }
        }
        return;
    }
    float* xr = x + (size_t)r * d;
    bool kv = true;
    if (rw.widx >= 0 && ct.hq) {
        // ---- NVFP4 residual cache: the row's codes against its cluster's block-entry centroid
        const size_t o = (size_t)rw.seq * sd.W_max + rw.widx;
        const float* ref = ct.z0 + ((size_t)rw.seq * ct.K + ct.labels[o]) * d;
        unsigned char* cq = ct.hq + o * (size_t)(d >> 1);
        unsigned char* cs = ct.hs + o * (size_t)(d >> 4);
        const bool patched = sd.within && patch[o] != 0;
        const bool fresh = !sd.within || patched;              // block entry records the row; a packet row replaces it
        const bool imposed = fresh && ct.fmask && ct.fmask[o];
        kv = fresh;
        const float* src = !sd.within ? xr : packet + o * d;
        const int n4 = d >> 2;
        float4 v[NORM_VPT];
        float ss = 0.f;
#pragma unroll
        for (int u = 0; u < NORM_VPT; ++u) {
            const int c4 = threadIdx.x + u * blockDim.x;
            const bool in = c4 < n4;
            const float4 rf = in ? __ldg(reinterpret_cast<const float4*>(ref) + c4) : make_float4(0.f, 0.f, 0.f, 0.f);
            v[u] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (u * (int)blockDim.x >= n4) continue;           // (the whole block is past the row)
            if (fresh) {
                const float4 raw = in ? __ldcg(reinterpret_cast<const float4*>(src) + c4) : make_float4(0.f, 0.f, 0.f, 0.f);
                unsigned cd, sb;
                float4 q = nvfp4_residual_chunk(raw, rf, &cd, &sb);
                if (in && imposed) {
                    cd = *reinterpret_cast<const unsigned short*>(ct.fq + o * (size_t)(d >> 1) + 2 * c4);
                    sb = ct.fs[o * (size_t)(d >> 4) + (c4 >> 2)];
                    q = nvfp4_dequant_chunk(cd, sb, rf);
                }
                if (in) {
                    *reinterpret_cast<unsigned short*>(cq + 2 * c4) = (unsigned short)cd;
                    if ((c4 & 3) == 0) cs[c4 >> 2] = (unsigned char)sb;
                    // a block-entry forward goes on with the plain row (only later steps read the cache); a refreshed
                    // row is what the cache now holds
                    v[u] = sd.within ? q : raw;
                }
            } else if (in) {
                v[u] = nvfp4_dequant_chunk(*reinterpret_cast<const unsigned short*>(cq + 2 * c4), cs[c4 >> 2], rf);
            }
            ss += v[u].x * v[u].x + v[u].y * v[u].y + v[u].z * v[u].z + v[u].w * v[u].w;
        }
        ss = block_sum(ss, red);
        const float inv = rsqrtf(ss / (float)d + eps);
#pragma unroll
        for (int u = 0; u < NORM_VPT; ++u) {
            const int c4 = threadIdx.x + u * blockDim.x;
            if (c4 < n4) {
                const float4 g = __ldg(reinterpret_cast<const float4*>(gain) + c4);
                store4<T>(a + 4 * c4, v[u].x * inv * g.x, v[u].y * inv * g.y, v[u].z * inv * g.z, v[u].w * inv * g.w);
                if (sd.within) reinterpret_cast<float4*>(xr)[c4] = v[u];
            }
        }
    } else if (rw.widx >= 0) {
        const size_t o = (size_t)rw.seq * sd.W_max + rw.widx;
        float* h = hc + o * d;
        if (sd.within) {
            // window row of a within-block step: the packet row if the previous layer selected it
            // (then it also replaces the cached hidden row), else the cached hidden row
            const bool patched = patch[o] != 0;
            kv = patched;
            norm_row<T>(patched ? packet + o * d : h, gain, eps, d, a, xr, patched ? h : nullptr, red);
        } else {
            norm_row<T>(xr, gain, eps, d, a, h, nullptr, red);      // block entry: record the hidden row
        }
    } else {
        norm_row<T>(xr, gain, eps, d, a, nullptr, nullptr, red);
    }
    if (threadIdx.x == 0) kvflag[r] = kv ? 1 : 0;
}
// Imposed NVFP4 codes written straight into the cache: one block per window row of one layer.
__global__ void impose_codes_kernel(const unsigned char* fmask, const unsigned char* fq, const unsigned char* fs, unsigned char* hq,
                                    unsigned char* hs, int d) {
    const size_t o = blockIdx.x;
    if (!fmask[o]) return;
    for (int i = threadIdx.x; i < (d >> 1); i += blockDim.x) hq[o * (size_t)(d >> 1) + i] = fq[o * (size_t)(d >> 1) + i];
    for (int i = threadIdx.x; i < (d >> 4); i += blockDim.x) hs[o * (size_t)(d >> 4) + i] = fs[o * (size_t)(d >> 4) + i];
}

template <typename T>
__global__ void prep_qkv_kernel(StepDesc sd, const Row* rows, float* x, float* hc, const float* packet,
                                const unsigned char* patch, const float* gain, float eps, int d,
                                T* a_out, unsigned char* kvflag, ClusterTabs ct) {
    KERNEL_PROLOGUE(3);   // prep_qkv_kernel
    __shared__ float red[33];
    prep_qkv_row<T>(sd, blockIdx.x, rows, x, hc, packet, patch, gain, eps, d, a_out, kvflag, red, ct);
}

// RMSNorm of a compacted list of rows (FFN input, LM-head input).
//   src row = list ? list[i] : i;  packet_rows: rows flagged as window rows read the packet
//   packet != null (steps whose down projection adds onto its output rows): the residual row of a selected window row is
//   also copied to its packet row, where that projection's parts then land
template <typename T>
__device__ __forceinline__ void prep_rows_row(int i, const float* x, const int* list, const int* m_count, const float* gain,
                                              float eps, int d, T* a_out, float* red, const Row* rows = nullptr,
                                              float* packet = nullptr, int W_max = 0) {
    T* a = a_out + (size_t)i * d;
    if (m_count && i >= *m_count) {
        for (int c = threadIdx.x; c < d; c += blockDim.x) a[c] = from_f<T>(0.f);
        return;
    }
    const int r = list ? list[i] : i;
    float* copy = nullptr;
    if (packet && rows) {
        const Row rw = rows[r];
        if (rw.pos >= 0 && rw.widx >= 0) copy = packet + ((size_t)rw.seq * W_max + rw.widx) * d;
    }
    norm_row<T>(x + (size_t)r * d, gain, eps, d, a, copy, nullptr, red);
}
template <typename T>
__global__ void prep_rows_kernel(const float* x, const int* list, const int* m_count, const float* gain,
                                 float eps, int d, T* a_out, const Row* rows, float* packet, int W_max) {
    KERNEL_PROLOGUE(4);   // prep_rows_kernel
    __shared__ float red[33];
    prep_rows_row<T>(blockIdx.x, x, list, m_count, gain, eps, d, a_out, red, rows, packet, W_max);
}

// LM-head input rows: entry i < n_act reads x[act_rows...]; later entries read packet rows.
struct HeadSrc { int kind; int index; };  // kind 0: x row `index`; 1: packet row `index` (= seq*W_max+w)
template <typename T>
__global__ void prep_head_kernel(const float* x, const float* packet, const HeadSrc* src_list,
                                 const int* m_count, const float* gain, float eps, int d, T* a_out) {
    KERNEL_PROLOGUE(5);   // prep_head_kernel
    __shared__ float red[33];
    const int i = blockIdx.x;
    T* a = a_out + (size_t)i * d;
    if (i >= *m_count) {
        for (int c = threadIdx.x; c < d; c += blockDim.x) a[c] = from_f<T>(0.f);
        return;
    }
    const HeadSrc hs = src_list[i];
    norm_row<T>((hs.kind ? packet : x) + (size_t)hs.index * d, gain, eps, d, a, nullptr, nullptr, red);
}

// Gather + RMSNorm for the stand-alone refresh kernel: row (s, i) <- h[s][idx[s][i]].
// The same launch also prepares what the projection behind it needs (one launch instead of four): the rotary entries
// of the row's position (rope_tab[pos][half], when rope_tab is given) and, in its first block, zeroed split-tile
// counters and status word of the caller's scratch.
template <typename T>
__global__ void prep_refresh_kernel(const T* h, const int* idx, const int* counts, int max_rows, int P,
                                    const float* gain, float eps, int d, T* a_out, float2* rope_tab, int half, double theta,
                                    int* counters, int n_counters, int* status) {
    KERNEL_PROLOGUE(6);   // prep_refresh_kernel
    __shared__ float red[33];
    const int m = blockIdx.x;
    const int s = m / max_rows, i = m - s * max_rows;
    T* a = a_out + (size_t)m * d;
    if (m == 0 && counters) {
        for (int c = threadIdx.x; c < n_counters; c += blockDim.x) counters[c] = 0;
        if (threadIdx.x == 0 && status) *status = 0;
    }
    if (i >= counts[s]) {
        for (int c = threadIdx.x; c < d; c += blockDim.x) a[c] = from_f<T>(0.f);
        return;
    }
    if (rope_tab) {
        const int pos = idx[s * max_rows + i];
        for (int k = threadIdx.x; k < half; k += blockDim.x) {
            const double ang = (double)pos * pow(theta, -(double)k / (double)half);
            rope_tab[(size_t)pos * half + k] = make_float2((float)cos(ang), (float)sin(ang));
        }
    }
    const T* src = h + ((size_t)s * P + idx[s * max_rows + i]) * d;
    float ss = 0.f;
    for (int c = threadIdx.x; c < d; c += blockDim.x) { const float v = to_f<T>(src[c]); ss += v * v; }
    ss = block_sum(ss, red);
    const float inv = rsqrtf(ss / (float)d + eps);
    for (int c = threadIdx.x; c < d; c += blockDim.x) a[c] = from_f<T>(to_f<T>(src[c]) * inv * gain[c]);
}

// ---------------------------------------------------------------------------------------
// Spherical K-means of the window's hidden rows at block entry (Sec. 4.1 "Cluster and Quantize Hidden States";
// Algorithm 1 "SphericalKMeans"), one CTA per sequence, and the cluster tables that follow from the labels.
// Deterministic reading: centre j starts at the unit vector of window row floor((j + 1/2) W / K); `iters` Lloyd
// iterations (assign to the largest cosine, lowest cluster on ties; centre = normalised sum of the members' unit
// vectors, an empty cluster keeps its centre); no more rows than clusters: every row its own cluster.
// All sums run in a fixed order.  K <= KM_MAX_K, W <= KM_MAX_W.
// ---------------------------------------------------------------------------------------
constexpr int KM_MAX_K = 16, KM_MAX_W = 1024, KM_THREADS = 512, KM_CL = 8, KM_SMEM_BYTES = 160 * 1024;
struct KmeansArgs {
    const float* x;            // entry forward: residual-stream rows of this layer [rows][d]
    int d, K, iters;
    int chunk;                 // columns of the centres staged in shared memory at a time (multiple of 128; K * chunk floats)
    int* labels; int* zpos; int* zcnt; int* members; int* moff;      // this layer's tables (see ClusterTabs)
    const int* forced_labels;  // [batch][W_max], first entry < 0: not forced (parity replay of another clustering)
    float* z0;                 // NVFP4 residual cache: [batch][K][d] member means of the plain rows (null: not kept)
    float* cent;               // scratch [batch][K * d + W_max]: the centres (member sums, not normalised), the rows' 1 / norm
};
// A cluster of KM_CL CTAs per sequence: the rows are split over the CTAs for the assignment, the columns for the
// centre update; cluster barriers (release / acquire) separate the phases, data of other CTAs is read through L2.
__device__ __forceinline__ void km_cluster_sync() {
    __syncthreads();
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__global__ void __cluster_dims__(KM_CL, 1, 1) __launch_bounds__(KM_THREADS) kmeans_kernel(StepDesc sd, KmeansArgs a) {
    KERNEL_PROLOGUE(18);   // kmeans_kernel
    extern __shared__ __align__(16) float Cs[];             // [K][chunk]
    const int KM_CHUNK = a.chunk;
    __shared__ float invn[KM_MAX_W];
    __shared__ int lab[KM_MAX_W];
    __shared__ float inv_c[KM_MAX_K];
    __shared__ int cnt[KM_MAX_K + 1], off[KM_MAX_K + 1];
    __shared__ unsigned short ord[KM_MAX_W];                 // window rows grouped by cluster, ascending inside a cluster
    const int s = blockIdx.y, rk = blockIdx.x, t = threadIdx.x, lane = t & 31, warp = t >> 5, nw = KM_THREADS / 32;
    const int W = sd.W, K = a.K, d = a.d;
    auto row = [&](int w) { return a.x + ((size_t)s * sd.rows_per_seq + (window_pos(sd, w) - sd.e0)) * d; };
    // lab[] -> cnt[], off[], ord[] (the whole block calls)
    auto group_rows = [&]() {
        __syncthreads();
        if (t < K) { int n = 0; for (int w = 0; w < W; ++w) n += lab[w] == t; cnt[t] = n; }
        __syncthreads();
        if (t == 0) { int o = 0; for (int j = 0; j < K; ++j) { off[j] = o; o += cnt[j]; } off[K] = o; }
        __syncthreads();
        if (t < K) { int o = off[t]; for (int w = 0; w < W; ++w) if (lab[w] == t) ord[o++] = (unsigned short)w; }
        __syncthreads();
    };
    float* C = a.cent + (size_t)s * ((size_t)K * d + sd.W_max);
    float* invn_g = C + (size_t)K * d;
    int* labels = a.labels + (size_t)s * sd.W_max;
    const int per = (W + KM_CL - 1) / KM_CL, w_lo = min(W, rk * per), w_hi = min(W, w_lo + per);     // this CTA's rows
    const int dper = (((d + KM_CL - 1) / KM_CL) + 3) & ~3, c_lo = min(d, rk * dper), c_hi = min(d, c_lo + dper);   // ... and columns
    const int* forced = a.forced_labels ? a.forced_labels + (size_t)s * sd.W_max : nullptr;
    if (forced && forced[0] >= 0) {
        for (int w = w_lo + t; w < w_hi; w += KM_THREADS) labels[w] = min(max(forced[w], 0), K - 1);
    } else if (W <= K) {
        for (int w = w_lo + t; w < w_hi; w += KM_THREADS) labels[w] = w;
    } else {
        for (int w = w_lo + warp; w < w_hi; w += nw) {
            float ss = 0.f;
            const float* h = row(w);
            for (int c = lane; c < d; c += 32) { const float v = h[c]; ss = fmaf(v, v, ss); }
            ss = warp_sum(ss);
            if (lane == 0) invn_g[w] = ss > 0.f ? rsqrtf(ss) : 0.f;
        }
        for (int j = rk; j < K; j += KM_CL) {                                  // starting centres: rows of the window
            const int w0 = (int)(((2 * j + 1) * (long long)W) / (2 * K));       // floor((j + 1/2) W / K)
            const float* h = row(w0);
            for (int c = t; c < d; c += KM_THREADS) C[(size_t)j * d + c] = h[c];
        }
        km_cluster_sync();
        for (int w = t; w < W; w += KM_THREADS) invn[w] = __ldcg(invn_g + w);
        for (int it = 0; it < a.iters; ++it) {
            // ---- assignment of this CTA's rows: a warp per row, the centres through shared memory in column chunks
            for (int w_base = w_lo; w_base < w_hi || w_base == w_lo; w_base += nw) {
                const int w = w_base + warp;
                const bool live = w < w_hi;
                const float* h = live ? row(w) : a.x;
                float dot[KM_MAX_K];
#pragma unroll
                for (int j = 0; j < KM_MAX_K; ++j) dot[j] = 0.f;
                float n2 = 0.f;                                                 // warp j: |centre j|^2 (first round only)
                for (int c0 = 0; c0 < d; c0 += KM_CHUNK) {
                    const int cw = min(KM_CHUNK, d - c0);
                    __syncthreads();
#pragma unroll 8
                    for (int e = t; e < K * (KM_CHUNK / 4); e += KM_THREADS) {
                        const int j = e / (KM_CHUNK / 4), q = e - j * (KM_CHUNK / 4);
                        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
                        if (4 * q < cw) v = __ldcg(reinterpret_cast<const float4*>(C + (size_t)j * d + c0) + q);
                        reinterpret_cast<float4*>(Cs + (size_t)j * KM_CHUNK)[q] = v;
                    }
                    __syncthreads();
                    if (w_base == w_lo && warp < K)
                        for (int q = lane; q < KM_CHUNK; q += 32) n2 = fmaf(Cs[warp * KM_CHUNK + q], Cs[warp * KM_CHUNK + q], n2);
                    if (live) {
#pragma unroll 4
                        for (int q = lane * 4; q < cw; q += 128) {
                            const float4 hv = *reinterpret_cast<const float4*>(h + c0 + q);
#pragma unroll
                            for (int j = 0; j < KM_MAX_K; ++j) {
                                if (j < K) {
                                    const float4 cv = *reinterpret_cast<const float4*>(Cs + j * KM_CHUNK + q);
                                    dot[j] = fmaf(hv.x, cv.x, fmaf(hv.y, cv.y, fmaf(hv.z, cv.z, fmaf(hv.w, cv.w, dot[j]))));
                                }
                            }
                        }
                    }
                }
                if (w_base == w_lo) {
                    n2 = warp_sum(n2);
                    if (warp < K && lane == 0) inv_c[warp] = n2 > 0.f ? rsqrtf(n2) : 0.f;
                }
                __syncthreads();
                if (live) {
                    float best = -INFINITY;
                    int bj = 0;
#pragma unroll
                    for (int j = 0; j < KM_MAX_K; ++j) {
                        if (j < K) {
                            const float cs = warp_sum(dot[j]) * inv_c[j] * invn[w];
                            if (cs > best) { best = cs; bj = j; }          // (lowest cluster on ties)
                        }
                    }
                    if (lane == 0) labels[w] = bj;
                }
                if (w_hi <= w_lo) break;
            }
            km_cluster_sync();
            if (it + 1 == a.iters) break;          // the centres of the last update are never used
            // ---- update of this CTA's columns: members added in ascending row order; an empty cluster keeps its centre
            for (int w = t; w < W; w += KM_THREADS) lab[w] = __ldcg(labels + w);
            group_rows();
            for (int c = c_lo + t; c < c_hi; c += KM_THREADS) {
                for (int j = 0; j < K; ++j) {
                    if (cnt[j] == 0) continue;
                    float acc = 0.f;
#pragma unroll 8
                    for (int i = off[j]; i < off[j + 1]; ++i) { const int w = ord[i]; acc += row(w)[c] * invn[w]; }
                    C[(size_t)j * d + c] = acc;
                }
            }
            km_cluster_sync();
        }
    }
    km_cluster_sync();
    // ---- tables: member counts, groups of members, rotary position of every proxy (first CTA); labels of the unused rows
    for (int w = t; w < W; w += KM_THREADS) lab[w] = __ldcg(labels + w);
    group_rows();
    if (rk == 0) {
        for (int w = W + t; w < sd.W_max; w += KM_THREADS) labels[w] = -1;
        if (t < K) {
            const int n = cnt[t];
            long long sp = 0;
            for (int i = off[t]; i < off[t + 1]; ++i) sp += window_pos(sd, ord[i]);
            a.zcnt[s * K + t] = n;
            a.zpos[s * K + t] = n > 0 ? (int)((2 * sp + n) / (2 * n)) : -1;       // floor(mean + 1/2)
        }
        if (t <= K) a.moff[s * (K + 1) + t] = off[t];
        for (int i = t; i < W; i += KM_THREADS) a.members[(size_t)s * sd.W_max + i] = ord[i];
    }
    if (a.z0) {
        // reference rows of the residual codec: the clusters' centroids as this block entry sees them (this CTA's columns)
        for (int c = c_lo + t; c < c_hi; c += KM_THREADS) {
            for (int j = 0; j < K; ++j) {
                float acc = 0.f;
#pragma unroll 8
                for (int i = off[j]; i < off[j + 1]; ++i) acc += row(ord[i])[c];
                a.z0[((size_t)s * K + j) * d + c] = cnt[j] > 0 ? acc * (1.f / (float)cnt[j]) : 0.f;
            }
        }
    }
}

// The codec on its own: codes, scales and stored values of rows x against reference rows ref (one CTA per row).
__global__ void nvfp4_residual_kernel(const float* x, const float* ref, int d, unsigned char* codes, unsigned char* scales, float* deq) {
    KERNEL_PROLOGUE(19);   // nvfp4_residual_kernel
    const size_t r = blockIdx.x;
    const int n4 = d >> 2;
    for (int c0 = 0; c0 < n4; c0 += blockDim.x) {
        const int c4 = c0 + threadIdx.x;
        const bool in = c4 < n4;
        const float4 v = in ? reinterpret_cast<const float4*>(x + r * d)[c4] : make_float4(0.f, 0.f, 0.f, 0.f);
        const float4 rf = in ? reinterpret_cast<const float4*>(ref + r * d)[c4] : make_float4(0.f, 0.f, 0.f, 0.f);
        unsigned cd, sb;
        const float4 q = nvfp4_residual_chunk(v, rf, &cd, &sb);
        if (in) {
            *reinterpret_cast<unsigned short*>(codes + r * (size_t)(d >> 1) + 2 * c4) = (unsigned short)cd;
            if ((c4 & 3) == 0) scales[r * (size_t)(d >> 4) + (c4 >> 2)] = (unsigned char)sb;
            reinterpret_cast<float4*>(deq + r * d)[c4] = q;
        }
    }
}

// ---------------------------------------------------------------------------------------
// Plain tiled GEMM on CUDA cores: out[m][n] = sum_k A[m][k] W[n][k], fp32 accumulate.
// 64x64 tile, 16-wide K slices, 256 threads, 4x4 outputs per thread.
// ---------------------------------------------------------------------------------------
template <typename T, int EPI>
__global__ void __launch_bounds__(256) gemm_simt_kernel(const T* __restrict__ A, const T* __restrict__ Wt,
                                                        int M, int Nout, int K, int w_tiled, EpiArgs e) {
    KERNEL_PROLOGUE(7);   // __launch_bounds__
    __shared__ float As[16][64 + 4];
    __shared__ float Ws[16][64 + 4];
    const int m0 = blockIdx.y * 64, n0 = blockIdx.x * 64;
    const int Mv = e.m_count ? min(M, *e.m_count) : M;
    if (m0 >= Mv) return;
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
    for (int k0 = 0; k0 < K; k0 += 16) {
        for (int t = threadIdx.x; t < 64 * 16; t += 256) {
            const int rr = t >> 4, kk = t & 15;
            const int m = m0 + rr, n = n0 + rr, k = k0 + kk;
            As[kk][rr] = (m < M && k < K) ? to_f<T>(A[(size_t)m * K + k]) : 0.f;
            // tile-major weights: block (n / 256, k / 64) is a contiguous [256][64] chunk
            const size_t wi = w_tiled ? ((size_t)((n >> 8) * (K >> 6) + (k >> 6)) << 14) + ((n & 255) << 6) + (k & 63)
                                      : (size_t)n * K + k;
            Ws[kk][rr] = (n < Nout && k < K) ? to_f<T>(Wt[wi]) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < 16; ++kk) {
            float a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
            for (int j = 0; j < 4; ++j) b[j] = Ws[kk][tx * 4 + j];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int m = m0 + ty * 4 + i;
        if (m >= Mv) continue;
#pragma unroll
        for (int j = 0; j < 4; j += 2) {
            const int n = n0 + tx * 4 + j;
            if (n + 1 < Nout) epilogue_pair<T, EPI>(e, m, n, acc[i][j], acc[i][j + 1]);
        }
    }
}

// ---------------------------------------------------------------------------------------
// Attention rows with drift, CUDA-core version: one warp per (row, head).
//   logp_j = s_j - logsumexp(s), s_j = q.k_j / sqrt(dh) over all N cache rows (Eq. 3, no mask);
//   out = sum_j p_j v_j;  recorded rows: kl = sum_j p_j (logp_j - prev_j), prev <- logp (Eq. 4).
// Dynamic shared memory: warps_per_block * N floats.
// ---------------------------------------------------------------------------------------
struct AttnArgs {
    const Row* rows; int n_rows;
    const void* q; const void* kc; const void* vc; void* out;
    // Stored attention rows: a row and one float per row such that log-probability = row - lse.  The tensor-core
    // kernel keeps scaled scores and their log-sum-exp; the other kernels keep log-probabilities and leave lse at 0.
    float* pprev;    // window rows: [batch][W_max][n_heads][N]   (null: none recorded)
    float* aprev;    // active rows: [batch][B][n_heads][N]       (null: none recorded)
    float* pprev_lse;   // [batch][W_max][n_heads]
    float* aprev_lse;   // [batch][B][n_heads]
    float* kl;       // [n_rows][n_heads]
    int N, n_heads, n_kv, head_dim, W_max, B, record_kl;
    int rows_per_seq, batch;   // layout of the forward's rows (stand-alone: n_rows, 1)
    float scale;
    int cluster_K;             // > 0: centroid proxies: pprev / pprev_lse hold [batch][cluster_K] proxy rows per head and
                               // window rows are not recorded
    int dirty_lo, dirty_hi;    // key positions [lo, hi) of every sequence that the kernel running just before may have
                               // written; all other K/V rows were complete before this forward was launched
    // stand-alone form: rows == null, row r belongs to sequence 0 and records into pprev[r]
};

template <typename T>
__global__ void attention_simt_kernel(AttnArgs a) {
    KERNEL_PROLOGUE(8);   // attention_simt_kernel
    extern __shared__ float sm[];
    const int wpb = blockDim.x >> 5, wid = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int r = blockIdx.x * wpb + wid, h = blockIdx.y;
    if (r >= a.n_rows) return;
    int seq = 0;
    float* prev = nullptr;
    if (a.rows) {
        const Row rw = a.rows[r];
        if (rw.pos < 0) return;
        seq = rw.seq;
        if (a.cluster_K > 0) {
            if (row_is_proxy(rw.widx) && a.pprev) prev = a.pprev + (((size_t)seq * a.cluster_K + row_cluster(rw.widx)) * a.n_heads + h) * a.N;
            else if (rw.aidx >= 0 && a.aprev) prev = a.aprev + (((size_t)seq * a.B + rw.aidx) * a.n_heads + h) * a.N;
        }
        else if (rw.widx >= 0 && a.pprev) prev = a.pprev + (((size_t)seq * a.W_max + rw.widx) * a.n_heads + h) * a.N;
        else if (rw.aidx >= 0 && a.aprev) prev = a.aprev + (((size_t)seq * a.B + rw.aidx) * a.n_heads + h) * a.N;
    } else if (a.pprev) {
        prev = a.pprev + ((size_t)r * a.n_heads + h) * a.N;
    }
    float* sc = sm + (size_t)wid * a.N;
    const int dh = a.head_dim, g = (h * a.n_kv) / a.n_heads;
    const int dq = a.n_heads * dh, dkv = a.n_kv * dh;
    const T* q = (const T*)a.q + (size_t)r * dq + h * dh;
    const T* K = (const T*)a.kc + (size_t)seq * a.N * dkv + g * dh;
    const T* V = (const T*)a.vc + (size_t)seq * a.N * dkv + g * dh;
    // scores
    float mx = -INFINITY;
    for (int j = lane; j < a.N; j += 32) {
        const T* kj = K + (size_t)j * dkv;
        float s = 0.f;
        for (int c = 0; c < dh; ++c) s = fmaf(to_f<T>(q[c]), to_f<T>(kj[c]), s);
        s *= a.scale;
        sc[j] = s;
        mx = fmaxf(mx, s);
    }
    mx = warp_max(mx);
    float sum = 0.f;
    for (int j = lane; j < a.N; j += 32) sum += expf(sc[j] - mx);
    sum = warp_sum(sum);
    const float lse = mx + logf(sum);
    float kl = 0.f;
    for (int j = lane; j < a.N; j += 32) {
        const float lp = sc[j] - lse;
        const float p = expf(lp);
        if (prev) {
            if (a.record_kl) kl += p * (lp - prev[j]);
            prev[j] = lp;
        }
        sc[j] = round_to<T>(p);
    }
    __syncwarp();
    if (a.kl) {
        kl = warp_sum(kl);
        if (lane == 0) a.kl[(size_t)r * a.n_heads + h] = (prev && a.record_kl) ? kl : 0.f;
    }
    if (a.out) {
        T* o = (T*)a.out + (size_t)r * dq + h * dh;
        for (int c = lane; c < dh; c += 32) {
            float acc = 0.f;
            for (int j = 0; j < a.N; ++j) acc = fmaf(sc[j], to_f<T>(V[(size_t)j * dkv + c]), acc);
            o[c] = from_f<T>(acc);
        }
    }
}

// ---------------------------------------------------------------------------------------
// Squared hidden-state change per row (Appendix B, Cor. 1): one warp per row, 128-bit loads.
// ---------------------------------------------------------------------------------------
template <typename T>
__global__ void hidden_delta_kernel(const T* __restrict__ a, const T* __restrict__ b, float* out, int rows, int d) {
    KERNEL_PROLOGUE(9);   // hidden_delta_kernel
    const int wpb = blockDim.x >> 5, wid = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int per = 16 / (int)sizeof(T);
    for (int r = blockIdx.x * wpb + wid; r < rows; r += gridDim.x * wpb) {
        const uint4* pa = reinterpret_cast<const uint4*>(a + (size_t)r * d);
        const uint4* pb = reinterpret_cast<const uint4*>(b + (size_t)r * d);
        float acc = 0.f;
        const int nv = d / per;
        for (int i = lane; i < nv; i += 32) {
            const uint4 ua = __ldg(pa + i), ub = __ldg(pb + i);
            const T* ea = reinterpret_cast<const T*>(&ua);
            const T* eb = reinterpret_cast<const T*>(&ub);
#pragma unroll
            for (int t = 0; t < per; ++t) { const float dd = to_f<T>(ea[t]) - to_f<T>(eb[t]); acc = fmaf(dd, dd, acc); }
        }
        for (int c = nv * per + lane; c < d; c += 32) {
            const float dd = to_f<T>(a[(size_t)r * d + c]) - to_f<T>(b[(size_t)r * d + c]);
            acc = fmaf(dd, dd, acc);
        }
        acc = warp_sum(acc);
        if (lane == 0) out[r] = acc;
    }
}

// ---------------------------------------------------------------------------------------
// Stale-row selection + compaction for one sequence (Sec. 4.1; Algorithm 1 "TopK").
// Block-wide radix select of the k-th largest drift, ties to the lower index, then a
// prefix-sum compaction to an ascending index list.  W <= SEL_MAX_W.
// ---------------------------------------------------------------------------------------
constexpr int SEL_THREADS = 1024;
constexpr int SEL_ITEMS = 4;
constexpr int SEL_MAX_W = SEL_THREADS * SEL_ITEMS;

struct SelSmem {
    int hist[256];
    int scan[33];
    unsigned prefix; int kleft; int total;
};

__device__ __forceinline__ unsigned float_key(float v) {   // order-preserving map to unsigned
    const unsigned u = __float_as_uint(v);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// D[i] valid for i < W.  Writes idx_out[0..count) ascending and (optional) flag_out[i] in {0,1}.
// Returns count (same value in every thread).  Must be called by all SEL_THREADS threads.
__device__ int select_one(const float* D, int W, int mode, int k, float thresh, float floor_,
                          int* idx_out, unsigned char* flag_out, SelSmem& s) {
    const int t = threadIdx.x;
    unsigned key[SEL_ITEMS];
    float val[SEL_ITEMS];
    bool cand[SEL_ITEMS], sel[SEL_ITEMS];
    // items are blocked: thread t owns indices t*ITEMS .. t*ITEMS+ITEMS-1 (keeps index order in scans)
#pragma unroll
    for (int u = 0; u < SEL_ITEMS; ++u) {
        const int i = t * SEL_ITEMS + u;
        const float v = i < W ? D[i] : 0.f;
        cand[u] = (i < W) && (v > floor_);          // NaN compares false: never a candidate
        val[u] = v;
        key[u] = float_key(v);
        sel[u] = false;
    }
    int ncand_local = 0;
#pragma unroll
    for (int u = 0; u < SEL_ITEMS; ++u) ncand_local += cand[u];
    int ncand;
    block_excl_scan(ncand_local, s.scan, &ncand);
    if (mode == 3) {                                  // ALL: every row
#pragma unroll
        for (int u = 0; u < SEL_ITEMS; ++u) sel[u] = (t * SEL_ITEMS + u) < W;
    } else if (mode == 2) {                           // THRESHOLD
#pragma unroll
        for (int u = 0; u < SEL_ITEMS; ++u) sel[u] = cand[u] && (val[u] > thresh);
    } else if (mode == 4 || k <= 0) {                 // NONE
    } else if (k >= ncand) {
#pragma unroll
        for (int u = 0; u < SEL_ITEMS; ++u) sel[u] = cand[u];
    } else {
        // radix select, most significant byte first
        if (t == 0) { s.prefix = 0u; s.kleft = k; }
        __syncthreads();
        for (int pass = 0; pass < 4; ++pass) {
            const int shift = 24 - 8 * pass;
            const unsigned himask = pass == 0 ? 0u : (0xFFFFFFFFu << (shift + 8));
            if (t < 256) s.hist[t] = 0;
            __syncthreads();
            const unsigned prefix = s.prefix;
#pragma unroll
            for (int u = 0; u < SEL_ITEMS; ++u)
                if (cand[u] && (key[u] & himask) == prefix) atomicAdd(&s.hist[(key[u] >> shift) & 255u], 1);
            __syncthreads();
            if (t == 0) {
                int left = s.kleft, bsel = 0;
                for (int bkt = 255; bkt >= 0; --bkt) {
                    const int c = s.hist[bkt];
                    if (c >= left) { bsel = bkt; break; }
                    left -= c;
                }
                s.kleft = left;
                s.prefix = prefix | ((unsigned)bsel << shift);
            }
            __syncthreads();
        }
        const unsigned kth = s.prefix;     // key of the k-th largest candidate
        const int need_eq = s.kleft;       // how many rows equal to it are taken (lowest indices)
        int eq_local = 0;
#pragma unroll
        for (int u = 0; u < SEL_ITEMS; ++u) eq_local += (cand[u] && key[u] == kth);
        int eq_total;
        int eq_before = block_excl_scan(eq_local, s.scan, &eq_total);
#pragma unroll
        for (int u = 0; u < SEL_ITEMS; ++u) {
            if (!cand[u]) continue;
            if (key[u] > kth) sel[u] = true;
            else if (key[u] == kth) { sel[u] = eq_before < need_eq; ++eq_before; }
        }
    }
    int nsel_local = 0;
#pragma unroll
    for (int u = 0; u < SEL_ITEMS; ++u) nsel_local += sel[u];
    int count;
    int off = block_excl_scan(nsel_local, s.scan, &count);
#pragma unroll
    for (int u = 0; u < SEL_ITEMS; ++u) {
        const int i = t * SEL_ITEMS + u;
        if (i < W && flag_out) flag_out[i] = sel[u] ? 1 : 0;
        if (sel[u]) idx_out[off++] = i;
    }
    __syncthreads();
    return count;
}

// Small windows (W <= SEL_SMALL_W, the in-step case: W = 3B): rank counting, two barriers.
// Thread i owns row i; rank = number of candidates ahead of it in (drift descending, index ascending) order.
constexpr int SEL_SMALL_W = 256;
// `i` = index of the calling thread among the participating threads (at least W of them); bar < 0: they are the
// whole block (__syncthreads), else they synchronise on named barrier `bar` with `nthr` threads.
__device__ __forceinline__ void sel_sync(int bar, int nthr) {
    if (bar < 0) __syncthreads();
    else asm volatile("bar.sync %0, %1;" ::"r"(bar), "r"(nthr) : "memory");
}
__device__ int select_small(const float* D, int W, int mode, int k, float thresh, float floor_,
                            int* idx_out, unsigned char* flag_out, int* sel_sh /* [SEL_SMALL_W] */,
                            int i = threadIdx.x, int bar = -1, int nthr = 0) {
    const float v = i < W ? D[i] : 0.f;
    const bool cand = i < W && v > floor_;
    bool sel = false;
    if (mode == 3) sel = i < W;
    else if (mode == 2) sel = cand && v > thresh;
    else if (mode != 4 && k > 0 && cand) {
        int rank = 0;
        for (int j = 0; j < W; ++j) {
            const float dj = D[j];
            rank += (dj > floor_ && (dj > v || (dj == v && j < i))) ? 1 : 0;
        }
        sel = rank < k;
    }
    if (i < SEL_SMALL_W) sel_sh[i] = sel ? 1 : 0;
    sel_sync(bar, nthr);
    int pos = 0, total = 0;
    for (int j = 0; j < W; ++j) { const int f = sel_sh[j]; total += f; pos += (j < i) ? f : 0; }
    if (i < W) {
        if (flag_out) flag_out[i] = sel ? 1 : 0;
        if (sel) idx_out[pos] = i;
    }
    sel_sync(bar, nthr);
    return total;
}

__global__ void __launch_bounds__(SEL_THREADS) select_kernel(const float* drift, int W, int mode, int k,
                                                             float thresh, float floor_, int* idx, int* count) {
    KERNEL_PROLOGUE(7);   // __launch_bounds__
    __shared__ SelSmem s;
    const int b = blockIdx.x;
    __shared__ int sel_sh[SEL_SMALL_W];
    const int c = W <= SEL_SMALL_W ? select_small(drift + (size_t)b * W, W, mode, k, thresh, floor_, idx + (size_t)b * W, nullptr, sel_sh)
                                   : select_one(drift + (size_t)b * W, W, mode, k, thresh, floor_, idx + (size_t)b * W, nullptr, s);
    if (threadIdx.x == 0) count[b] = c;
}

// In-step selection for every refreshing sequence, plus the compacted row list of the sparse
// forward: all valid non-window rows followed by the selected window rows.
struct StepSelArgs {
    const float* kl;            // [rows][n_heads] per-head drift of the forward's rows
    float* drift;               // [batch][W_max] (output, this layer)
    int* sel_idx; int* sel_cnt; // this layer: [batch][W_max], [batch]
    unsigned char* flag_next;   // patch flags of the next layer [batch][W_max]
    const int* forced_idx; const int* forced_cnt;   // this layer (cnt < 0: not forced)
    int* list; int* list_count; // compacted rows of the sparse forward
    int* stats;                 // [0] += refreshed rows
    int n_heads, mode, k, W_max;
    float thresh, floor_;
    ClusterTabs ct;             // centroid proxies (ct.K > 0): drift per cluster, the top cluster_k clusters' members
    int cluster_k;
};

// The same work for a batch of one sequence with a window of at most SEL_SMALL_W rows, done by `nthr` >= W threads
// (t = 0 .. nthr-1) of a kernel that is busy otherwise: they synchronise on named barrier `bar` only.  Used by
// the O projection, whose idle warps select the stale rows while the weights stream.
__device__ __forceinline__ void step_select_inline(const StepDesc& sd, const StepSelArgs& a, int t, int nthr, int bar,
                                                   float* dsh /* [SEL_SMALL_W] */, int* sel_sh /* [SEL_SMALL_W] */) {
    int cnt = 0;
    int* idx = a.sel_idx;
    if (sd.refresh.v[0]) {
        for (int w0 = 0; w0 < sd.W; w0 += nthr / 8) {
            const int w = w0 + (t >> 3), part = t & 7;
            float acc = 0.f;
            if (w < sd.W) {
                const float* kr = a.kl + (size_t)(sd.B + w) * a.n_heads;
                for (int h = part; h < a.n_heads; h += 8) acc += __ldcg(kr + h);
            }
            acc += __shfl_xor_sync(0xffffffffu, acc, 1);
            acc += __shfl_xor_sync(0xffffffffu, acc, 2);
            acc += __shfl_xor_sync(0xffffffffu, acc, 4);
            if (w < sd.W && part == 0) {
                const float dv = acc / (float)a.n_heads;
                dsh[w] = dv;
                a.drift[w] = dv;
            }
        }
        sel_sync(bar, nthr);
        unsigned char* fl = a.flag_next;
        const int fc = a.forced_cnt ? a.forced_cnt[0] : -1;
        if (fc >= 0) {
            for (int w = t; w < sd.W; w += nthr) fl[w] = 0;
            sel_sync(bar, nthr);
            for (int i = t; i < fc; i += nthr) { const int w = a.forced_idx[i]; idx[i] = w; fl[w] = 1; }
            cnt = fc;
            sel_sync(bar, nthr);
        } else {
            cnt = select_small(dsh, sd.W, a.mode, a.k, a.thresh, a.floor_, idx, fl, sel_sh, t, bar, nthr);
        }
    }
    // compacted row list of the sparse forward: the active rows, then the selected window rows
    for (int i = t; i < sd.B; i += nthr) a.list[i] = i;
    for (int i = t; i < cnt; i += nthr) a.list[sd.B + i] = sd.B + idx[i];
    if (t == 0) {
        a.sel_cnt[0] = cnt;
        *a.list_count = sd.B + cnt;
        atomicAdd(a.stats, cnt);
    }
}

// One CTA per sequence; the CTA that finishes last (arrival counter a.stats[3], left at zero again) builds the
// compacted row list from all sequences' selections.
__global__ void __launch_bounds__(SEL_THREADS) step_select_kernel(StepDesc sd, StepSelArgs a) {
    KERNEL_PROLOGUE(7);   // __launch_bounds__
    __shared__ SelSmem s;
    __shared__ float dsh[SEL_MAX_W > 1024 ? 1024 : SEL_MAX_W];
    __shared__ int sel_sh[SEL_SMALL_W];
    __shared__ int offs[65];
    __shared__ int last_sh;
    const int t = threadIdx.x;
    const int sq = blockIdx.x;
    int cnt = 0;
    if (sd.refresh.v[sq] && a.ct.K > 0) {
        // ---- centroid proxies (Sec. 4.1; Algorithm 1 "KL", "TopK", M[K]): drift of the K proxy rows, the
        // cluster_k clusters with the largest drift, then their member rows in ascending order
        __shared__ int csel[KM_MAX_K], ctmp[KM_MAX_K];
        const int K = a.ct.K;
        if (t < K) {
            const float* kr = a.kl + (size_t)(sq * sd.rows_per_seq + sd.B + sd.W + t) * a.n_heads;
            float acc = 0.f;
            for (int h = 0; h < a.n_heads; ++h) acc += __ldg(kr + h);
            const float dv = a.ct.zcnt[sq * K + t] > 0 ? acc / (float)a.n_heads : 0.f;       // an empty cluster never drifts
            dsh[t] = dv;
            a.drift[sq * a.W_max + t] = dv;
        }
        __syncthreads();
        int* idx = a.sel_idx + sq * a.W_max;
        unsigned char* fl = a.flag_next + sq * a.W_max;
        const int fc = a.forced_cnt ? a.forced_cnt[sq] : -1;
        if (fc >= 0) {
            for (int w = t; w < sd.W; w += blockDim.x) fl[w] = 0;
            __syncthreads();
            for (int i = t; i < fc; i += blockDim.x) { const int w = a.forced_idx[sq * a.W_max + i]; idx[i] = w; fl[w] = 1; }
            cnt = fc;
        } else {
            select_small(dsh, K, 1 /* top-k count */, a.cluster_k, a.thresh, a.floor_, ctmp, nullptr, sel_sh);
            if (t < K) csel[t] = sel_sh[t];
            __syncthreads();
            const bool sel = t < sd.W && csel[a.ct.labels[(size_t)sq * a.W_max + t]] != 0;
            if (t < SEL_SMALL_W) sel_sh[t] = sel ? 1 : 0;
            __syncthreads();
            int pos = 0, total = 0;
            for (int j = 0; j < sd.W; ++j) { const int f = sel_sh[j]; total += f; pos += (j < t) ? f : 0; }
            if (t < sd.W) { fl[t] = sel ? 1 : 0; if (sel) idx[pos] = t; }
            cnt = total;
        }
    } else if (sd.refresh.v[sq]) {
        // head mean of the per-head drift (Eq. 4): eight lanes per row, all loads of a row in flight at once;
        // the partial sums are combined in a fixed order
        for (int w0 = 0; w0 < sd.W; w0 += blockDim.x / 8) {
            const int w = w0 + (t >> 3), part = t & 7;
            float acc = 0.f;
            if (w < sd.W) {
                const float* kr = a.kl + (size_t)(sq * sd.rows_per_seq + sd.B + w) * a.n_heads;
                for (int h = part; h < a.n_heads; h += 8) acc += __ldg(kr + h);
            }
            acc += __shfl_xor_sync(0xffffffffu, acc, 1);
            acc += __shfl_xor_sync(0xffffffffu, acc, 2);
            acc += __shfl_xor_sync(0xffffffffu, acc, 4);
            if (w < sd.W && part == 0) {
                const float dv = acc / (float)a.n_heads;
                dsh[w] = dv;
                a.drift[sq * a.W_max + w] = dv;
            }
        }
        __syncthreads();
        int* idx = a.sel_idx + sq * a.W_max;
        unsigned char* fl = a.flag_next + sq * a.W_max;
        const int fc = a.forced_cnt ? a.forced_cnt[sq] : -1;
        if (fc >= 0) {
            for (int w = t; w < sd.W; w += blockDim.x) fl[w] = 0;
            __syncthreads();
            for (int i = t; i < fc; i += blockDim.x) { const int w = a.forced_idx[sq * a.W_max + i]; idx[i] = w; fl[w] = 1; }
            cnt = fc;
        } else {
            cnt = sd.W <= SEL_SMALL_W ? select_small(dsh, sd.W, a.mode, a.k, a.thresh, a.floor_, idx, fl, sel_sh)
                                      : select_one(dsh, sd.W, a.mode, a.k, a.thresh, a.floor_, idx, fl, s);
        }
    }
    __syncthreads();
    if (t == 0) {
        a.sel_cnt[sq] = cnt;
        int last = 1;
        if (sd.batch > 1) {
            __threadfence();
            last = atomicAdd(a.stats + 3, 1) == sd.batch - 1;
            __threadfence();
        }
        last_sh = last;
    }
    __syncthreads();
    if (!last_sh) return;
    // compacted row list of the sparse forward: all active rows (row id = s*rows_per_seq + j), then the selected
    // window rows sequence by sequence
    const int nb = sd.batch * sd.B;
    if (t == 0) {
        int base = nb;
        for (int q = 0; q < sd.batch; ++q) { offs[q] = base; base += __ldcg(a.sel_cnt + q); }
        offs[sd.batch] = base;
        *a.list_count = base;
        atomicAdd(a.stats, base - nb);
        a.stats[3] = 0;
    }
    for (int i = t; i < nb; i += blockDim.x) a.list[i] = (i / sd.B) * sd.rows_per_seq + (i % sd.B);
    __syncthreads();
    for (int q = 0; q < sd.batch; ++q) {
        const int b0 = offs[q], n = offs[q + 1] - b0;
        for (int i = t; i < n; i += blockDim.x) a.list[b0 + i] = q * sd.rows_per_seq + sd.B + __ldcg(a.sel_idx + q * a.W_max + i);
    }
}

// ---------------------------------------------------------------------------------------
// LM-head row list: every active row, then (refresh steps with suffix commit) the rows the last
// layer selected that lie in the suffix window and are still masked (Sec. 4.2 "Suffix Block Commit")
// ---------------------------------------------------------------------------------------
__global__ void build_head_list_kernel(StepDesc sd, const int* y, int mask_id, const int* sel_idx,
                                       const int* sel_cnt, int use_suffix, int act_row0_stride,
                                       HeadSrc* list, int* count, int* suf_seq, int* suf_w) {
    KERNEL_PROLOGUE(10);   // build_head_list_kernel
    // act_row0_stride: forward row of active j in sequence s = s*rows_per_seq + (act offset) + j
    const int t = threadIdx.x;
    const int nb = sd.batch * sd.B;
    const int act_off = sd.kind == 2 ? 0 : (sd.act_start - sd.e0);
    for (int i = t; i < nb; i += blockDim.x) {
        HeadSrc h; h.kind = 0; h.index = (i / sd.B) * sd.rows_per_seq + act_off + (i % sd.B);
        list[i] = h;
    }
    __syncthreads();
    if (t == 0) {
        int n = nb;
        if (use_suffix) {
            for (int s = 0; s < sd.batch; ++s) {
                if (!sd.refresh.v[s]) continue;
                const int c = sel_cnt[s];
                for (int i = 0; i < c; ++i) {
                    const int w = sel_idx[s * sd.W_max + i];
                    if (w < sd.n_pre) continue;
                    const int pos = window_pos(sd, w);
                    if (y[s * sd.N + pos] != mask_id) continue;
                    HeadSrc h; h.kind = 1; h.index = s * sd.W_max + w;
                    list[n] = h; suf_seq[n - nb] = s; suf_w[n - nb] = w;
                    ++n;
                }
            }
        }
        *count = n;
    }
    (void)act_row0_stride;
}

// ---------------------------------------------------------------------------------------
// Confidence of logits rows (Eq. 1 and the confidence of Sec. 2): two stages.
// ---------------------------------------------------------------------------------------
struct ConfPart { float mx_all; float sum; float mx_ex; int arg_ex; };

__global__ void conf_partial_kernel(const float* logits, const int* m_count, int rows, int V, int mask_id,
                                    int chunks, ConfPart* part) {
    KERNEL_PROLOGUE(11);   // conf_partial_kernel
    __shared__ float red[33];
    __shared__ float bv[32];
    __shared__ int bi[32];
    const int r = blockIdx.y, ch = blockIdx.x;
    if (r >= rows || (m_count && r >= *m_count)) return;
    const int per = ((V + chunks - 1) / chunks + 3) & ~3;
    const int v0 = ch * per, v1 = min(V, v0 + per);
    const float* l = logits + (size_t)r * V;
    // one pass: every thread keeps a running (max, sum of exp relative to that max) and its best
    // non-[MASK] candidate; 128-bit loads when the row is 16-byte aligned
    float mx = -INFINITY, sum = 0.f, mxe = -INFINITY;
    int arg = 0x7fffffff;
    if ((V & 3) == 0) {
        const float4* l4 = reinterpret_cast<const float4*>(l);
        for (int v4 = (v0 >> 2) + threadIdx.x; v4 < (v1 >> 2); v4 += blockDim.x) {
            const float4 x = __ldg(l4 + v4);
            const float xs[4] = {x.x, x.y, x.z, x.w};
            const float m4 = fmaxf(fmaxf(x.x, x.y), fmaxf(x.z, x.w));
            const float nm = fmaxf(mx, m4);
            sum = sum * expf(mx - nm) + expf(x.x - nm) + expf(x.y - nm) + expf(x.z - nm) + expf(x.w - nm);
            mx = nm;
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int v = 4 * v4 + u;
                if (v != mask_id && (xs[u] > mxe || (xs[u] == mxe && v < arg))) { mxe = xs[u]; arg = v; }
            }
        }
    } else {
        for (int v = v0 + threadIdx.x; v < v1; v += blockDim.x) {
            const float x = l[v];
            const float nm = fmaxf(mx, x);
            sum = sum * expf(mx - nm) + expf(x - nm);
            mx = nm;
            if (v != mask_id && (x > mxe || (x == mxe && v < arg))) { mxe = x; arg = v; }
        }
    }
    const float bmx = block_max(mx, red);
    sum = (mx == -INFINITY) ? 0.f : sum * expf(mx - bmx);
    sum = block_sum(sum, red);
    // argmax with lowest id on ties
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, mxe, o);
        const int oi = __shfl_xor_sync(0xffffffffu, arg, o);
        if (ov > mxe || (ov == mxe && oi < arg)) { mxe = ov; arg = oi; }
    }
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = blockDim.x >> 5;
    if (lane == 0) { bv[wid] = mxe; bi[wid] = arg; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < nw; ++w)
            if (bv[w] > mxe || (bv[w] == mxe && bi[w] < arg)) { mxe = bv[w]; arg = bi[w]; }
        ConfPart p; p.mx_all = bmx; p.sum = (v1 > v0) ? sum : 0.f; p.mx_ex = mxe; p.arg_ex = arg;
        part[(size_t)r * chunks + ch] = p;
    }
}

__global__ void conf_final_kernel(const ConfPart* part, const int* m_count, int rows, int chunks,
                                  int* yhat, float* conf) {
    KERNEL_PROLOGUE(12);   // conf_final_kernel
    const int r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= rows || (m_count && r >= *m_count)) return;
    const ConfPart* p = part + (size_t)r * chunks;
    float mx = -INFINITY, mxe = -INFINITY;
    int arg = 0x7fffffff;
    for (int c = 0; c < chunks; ++c) {
        mx = fmaxf(mx, p[c].mx_all);
        if (p[c].mx_ex > mxe || (p[c].mx_ex == mxe && p[c].arg_ex < arg)) { mxe = p[c].mx_ex; arg = p[c].arg_ex; }
    }
    float sum = 0.f;
    for (int c = 0; c < chunks; ++c)
        if (p[c].sum > 0.f) sum += p[c].sum * expf(p[c].mx_all - mx);
    yhat[r] = arg;
    conf[r] = expf(mxe - mx) / sum;
}

// ---------------------------------------------------------------------------------------
// Commit rule (Sec. 4.2; Algorithm 1 after the layer loop; Eq. 2): one block per sequence.
// ---------------------------------------------------------------------------------------
struct CommitArgs {
    int* y;                      // [batch][N]
    const float* conf; const int* yhat;   // LM rows: active rows first ([batch*B]), then suffix rows
    const float* kl;             // per-head drift of the forward's rows (last layer) [rows][n_heads]
    float* delta_out;            // [batch][B]
    float* Delta_out; float* taud_out;
    float* theta; int* theta_cnt;   // [batch][hist][B] ring, [batch] number pushed so far
    int* commit_flags;           // [batch][B]
    int* own_flags;              // [batch][B]: the rule's own decision, before a forced decision replaces it
    int* suffix_flags;           // [batch][W_max]
    const int* head_count; const int* suf_seq; const int* suf_w;
    const int* forced_pos; int forced_n;      // [batch][forced_n] absolute positions, -1 unused (null: free-running)
    const int* forced_tok;                    // optional tokens written at the forced positions (null: own prediction)
    int* seq_info;               // [batch][8]: committed, by_conf, by_drift, by_quota, suffix, eos, masked_left, nonfinite;
                                 // then 8 more words: the step's counters (stats[0..3]) and the GEMM status word
    const int* stats; const int* status; int batch;
    int n_heads, hist, mask_id, eos_id, act_row_off, steps_used, steps_per_block, use_drift, use_suffix, ge;
    float tau_s, alpha, tau_suffix;
};

__global__ void commit_kernel(StepDesc sd, CommitArgs a) {
    KERNEL_PROLOGUE(13);   // commit_kernel
    __shared__ float s_conf[256];
    __shared__ unsigned char s_masked[256], s_flag[256];
    __shared__ int cnt[8];
    const int s = blockIdx.x, j = threadIdx.x, B = sd.B;
    if (j < 8) cnt[j] = 0;
    __syncthreads();
    const bool within = sd.record_kl != 0;
    float c = 0.f, dl = 0.f, Dl = 0.f, td = 0.f;
    int tok = 0, yh = 0;
    bool masked = false;
    int flag = 0;
    if (j < B) {
        tok = a.y[s * sd.N + sd.act_start + j];
        masked = tok == a.mask_id;
        c = a.conf[s * B + j];
        yh = a.yhat[s * B + j];
        if (within) {
            dl = a.delta_out[s * B + j];      // written by delta_kernel at the end of the forward
            const int pushed = a.theta_cnt[s];
            const int nh = min(pushed, a.hist);
            float mean = 0.f;
            if (nh > 0) {
                // oldest to newest, like a running list
                for (int u = 0; u < nh; ++u) mean += a.theta[((size_t)s * a.hist + ((pushed - nh + u) % a.hist)) * B + j];
                mean /= (float)nh;
            }
            Dl = dl - mean;
            if (a.hist > 0) a.theta[((size_t)s * a.hist + (pushed % a.hist)) * B + j] = dl;
        }
        td = a.alpha * (a.tau_s - c) * (a.tau_s - c);
        if (masked) {
            if (!(c == c)) atomicAdd(&cnt[7], 1);
            const bool c_ok = a.ge ? (c >= a.tau_s) : (c > a.tau_s);
            const bool d_ok = within && a.use_drift && (a.ge ? (Dl >= td) : (Dl > td));
            if (c_ok) flag = 1 | 2;
            else if (d_ok) flag = 1 | 4;
        }
        a.delta_out[s * B + j] = dl;
        a.Delta_out[s * B + j] = Dl;
        a.taud_out[s * B + j] = td;
        s_conf[j] = c; s_masked[j] = masked; s_flag[j] = (unsigned char)flag;
        if (masked) atomicAdd(&cnt[6], 1);
        if (flag) atomicAdd(&cnt[0], 1);
    }
    __syncthreads();
    if (j == 0 && within && a.hist > 0) a.theta_cnt[s] = a.theta_cnt[s] + 1;
    const int n_masked = cnt[6];
    {
        // quota top-up: the most confident masked rows not yet committed (ties: lowest position)
        const int denom = max(1, a.steps_per_block - a.steps_used);
        const int quota = n_masked > 0 ? (n_masked + denom - 1) / denom : 0;
        const int need = quota - cnt[0];
        if (need > 0 && j < B && masked && !flag) {
            int rank = 0;
            for (int u = 0; u < B; ++u)
                if (s_masked[u] && !s_flag[u] && (s_conf[u] > c || (s_conf[u] == c && u < j))) ++rank;
            if (rank < need) flag = 1 | 8;
        }
    }
    if (j < B) a.own_flags[s * B + j] = flag;
    if (a.forced_pos) {
        // a forced decision replaces the rule's own (kept in own_flags); the label of a row the rule also chose stays
        if (j < B) {
            const int own = flag;
            flag = 0;
            const int pos = sd.act_start + j;
            for (int u = 0; u < a.forced_n; ++u)
                if (a.forced_pos[s * a.forced_n + u] == pos) {
                    flag = own ? own : (1 | 8);
                    if (a.forced_tok) yh = a.forced_tok[s * a.forced_n + u];
                }
            if (!masked) flag = 0;
        }
    }
    __syncthreads();
    if (j < 6) cnt[j] = 0;
    __syncthreads();
    if (j < B) {
        a.commit_flags[s * B + j] = flag;
        if (flag & 1) {
            a.y[s * sd.N + sd.act_start + j] = yh;
            atomicAdd(&cnt[0], 1);
            if (flag & 2) atomicAdd(&cnt[1], 1);
            if (flag & 4) atomicAdd(&cnt[2], 1);
            if (flag & 8) atomicAdd(&cnt[3], 1);
            if (yh == a.eos_id) atomicAdd(&cnt[5], 1);
        }
    }
    // suffix rows of the final packet: confidence alone decides
    for (int w = j; w < sd.W_max; w += blockDim.x) a.suffix_flags[s * sd.W_max + w] = 0;
    __syncthreads();
    if (a.use_suffix && within) {
        const int n_suf = *a.head_count - sd.batch * B;
        for (int i = j; i < n_suf; i += blockDim.x) {
            if (a.suf_seq[i] != s) continue;
            const int w = a.suf_w[i];
            const int pos = window_pos(sd, w);
            const float sc = a.conf[sd.batch * B + i];
            bool ok = a.ge ? (sc >= a.tau_suffix) : (sc > a.tau_suffix);
            int t2 = a.yhat[sd.batch * B + i];
            int f = 1 | (ok ? 4 : 0);          // bit 2: the rule's own decision for this eligible row
            if (a.forced_pos) {
                ok = false;
                for (int u = 0; u < a.forced_n; ++u)
                    if (a.forced_pos[s * a.forced_n + u] == pos) { ok = true; if (a.forced_tok) t2 = a.forced_tok[s * a.forced_n + u]; }
            }
            if (ok && a.y[s * sd.N + pos] == a.mask_id) {
                a.y[s * sd.N + pos] = t2;
                f |= 2;
                atomicAdd(&cnt[0], 1); atomicAdd(&cnt[4], 1);
                if (t2 == a.eos_id) atomicAdd(&cnt[5], 1);
            }
            a.suffix_flags[s * sd.W_max + w] = f;
        }
    }
    __syncthreads();
    if (j == 0) {
        int* o = a.seq_info + s * 8;
        o[0] = cnt[0]; o[1] = cnt[1]; o[2] = cnt[2]; o[3] = cnt[3]; o[4] = cnt[4]; o[5] = cnt[5];
        o[6] = n_masked - (cnt[0] - cnt[4]);
        o[7] = cnt[7];
        if (s == 0) {        // one record for the host: a single copy brings everything the controller reads
            int* t = a.seq_info + a.batch * 8;
            t[0] = a.stats[0]; t[1] = a.stats[1]; t[2] = a.stats[2]; t[3] = a.stats[3];
            t[4] = *a.status;
        }
    }
}

// Last-layer drift of the active rows (Algorithm 1, delta): mean over heads of the per-head KL.
__global__ void delta_kernel(StepDesc sd, const float* kl, int act_row_off, int n_heads, float* delta) {
    KERNEL_PROLOGUE(14);   // delta_kernel
    const int s = blockIdx.x, j = threadIdx.x;
    if (j >= sd.B) return;
    float dl = 0.f;
    if (sd.record_kl) {
        const float* kr = kl + (size_t)(s * sd.rows_per_seq + act_row_off + j) * n_heads;
        float acc = 0.f;
        for (int h = 0; h < n_heads; ++h) acc += kr[h];
        dl = acc / (float)n_heads;
    }
    delta[s * sd.B + j] = dl;
}

// gather rows of x into a keep buffer: dst[s][j][:] = x[row(s, j)][:]
__global__ void keep_hidden_kernel(StepDesc sd, const float* x, int act_row_off, int d, float* dst) {
    KERNEL_PROLOGUE(15);   // keep_hidden_kernel
    const int i = blockIdx.x;
    const int s = i / sd.B, j = i - s * sd.B;
    const float* src = x + (size_t)(s * sd.rows_per_seq + act_row_off + j) * d;
    float* o = dst + (size_t)i * d;
    for (int c = threadIdx.x; c < d; c += blockDim.x) o[c] = src[c];
}

// y = [prompt ; MASK ...] from a prompt that already lives on the device (ids clamped to the vocabulary)
__global__ void init_tokens_kernel(int* y, const int* prompt, int batch, int prompt_len, int N, int mask_id, int vocab) {
    KERNEL_PROLOGUE(16);   // init_tokens_kernel
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= batch * N) return;
    const int s = i / N, pos = i - s * N;
    int t = mask_id;
    if (pos < prompt_len) {
        t = prompt[s * prompt_len + pos];
        t = t < 0 ? 0 : (t >= vocab ? vocab - 1 : t);
        if (t == mask_id) t = (mask_id + 1) % vocab;
    }
    y[i] = t;
}

// rotary table: tab[pos][i] = (cos, sin)(pos * theta^(-2i/dh)), computed in double precision
__global__ void rope_table_kernel(float2* tab, int N, int half, double theta) {
    KERNEL_PROLOGUE(17);   // rope_table_kernel
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= N * half) return;
    const int pos = i / half, k = i - pos * half;
    const double inv = pow(theta, -(double)k / (double)half);
    const double ang = (double)pos * inv;
    tab[i] = make_float2((float)cos(ang), (float)sin(ang));
}

}  // namespace ps
