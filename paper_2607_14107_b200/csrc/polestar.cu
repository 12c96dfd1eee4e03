// Host side of the Polestar C ABI: workspace plan, controller (Algorithm 1's outer loops and
// the update schedule of Sec. 4.1), kernel sequencing of one forward, read-back.
#include "../../include/polestar.h"

#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <climits>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <atomic>
#include <map>
#include <mutex>
#include <new>
#include <tuple>
#include <vector>

#include "attn_mma.cuh"
#include "gemm_tc.cuh"
#include "attn_tc.cuh"
#include "attn_stream.cuh"
#include "gemm_chain.cuh"
#include "kernels.cuh"

using namespace ps;

#define CK(call)                                             \
    do {                                                     \
        cudaError_t _e = (call);                             \
        if (_e != cudaSuccess) { last_cuda_error = _e; return POLESTAR_E_CUDA; } \
    } while (0)

static thread_local cudaError_t last_cuda_error = cudaSuccess;

// ------------------------------------------------------------------------------------------
// environment switches: read by polestar_init (into the context) and by polestar_reload_env,
// never on the launch path
// ------------------------------------------------------------------------------------------
struct Switches {
    int pdl = 1;             // POLESTAR_PDL: programmatic dependent launch between the kernels of a forward
    int evict_first = 1;     // POLESTAR_GEMM_EVICT_FIRST: weight TMA loads carry the evict_first L2 policy
    int fuse_select = 1;     // POLESTAR_FUSE_SELECT: batch-1 selection inside the O projection
    int chain = 1;           // POLESTAR_CHAIN: O -> norm -> gate/up -> down as one persistent launch
    int stages = 0;          // POLESTAR_GEMM_STAGES: operand ring depth (0 = 3 for one token tile, else 4)
    int align_pct = 85;      // POLESTAR_GEMM_ALIGN_PCT
    int half_align = 1;      // POLESTAR_GEMM_HALF_ALIGN
    int attn_kernel = 0;     // POLESTAR_ATTN_KERNEL: 0 automatic, else force a kernel variant
    int attn_simt = 0;       // POLESTAR_ATTN_SIMT: CUDA-core attention for bf16 models (debugging)
    int refresh_simt = 0;    // POLESTAR_REFRESH_SIMT
    int fuse_prep = 0;       // POLESTAR_FUSE_PREP (measured negative result, kept with its test)
    int fold_norm = 0;       // POLESTAR_FOLD_NORM (same)
    int tall_rows = 2048;    // POLESTAR_GEMM_TALL_ROWS: projections of at least this many rows use 256-token CTA tiles
                             // (measured on the 4096-wide QKV projection alone: 4096 rows 0.72 -> 0.75 of the bf16 peak, 8192
                             // rows 0.70 -> 0.79, 16384 rows 0.66 -> 0.78, 2048 rows 0.67 -> 0.64, 1024 rows 0.56 -> 0.51; in
                             // the long-generation decode, whose refresh steps have 2048 rows, 335 -> 339 tokens/s with the
                             // threshold at 2048, no change at 512)
    int tall_rows_ffn = 512; // POLESTAR_GEMM_TALL_ROWS_FFN: the same threshold for the gate/up projection, whose epilogue is short
                             // enough for the tall tile to pay from 512 rows on (follows POLESTAR_GEMM_TALL_ROWS when only that is set)
    int one_tall = 1;        // POLESTAR_GEMM_ONE_TALL: projections of 129 - 256 rows run as one 256-token tile
    int accumulate = 1;      // POLESTAR_GEMM_ACCUMULATE: O / down projections of the chained kernel add their parts onto
                             // the residual rows in L2 (0: ordered reduction of published partial tiles, bit-reproducible)
    int chain_qkv = 0;       // POLESTAR_CHAIN_QKV (same)
    int pair_rows = 1 << 30; // POLESTAR_GEMM_PAIR_ROWS: projections of at least this many rows run on CTA pairs (tcgen05 cta_group::2)
    int epi_groups = 3;      // POLESTAR_GEMM_EPI_GROUPS: groups of four warps that drain an accumulator when a projection
                             // has several token tiles (1: the four epilogue warps alone)
    int l2promo = (int)CU_TENSOR_MAP_L2_PROMOTION_L2_128B;   // POLESTAR_TMA_L2PROMO
    int gemm_trace = -1;     // POLESTAR_GEMM_TRACE (POLESTAR_TRACE builds)
    int kernel_trace = 0;    // POLESTAR_KERNEL_TRACE (POLESTAR_TRACE builds)
};
static int env_int(const char* name, int dflt) {
    const char* s = getenv(name);
    return s ? atoi(s) : dflt;
}
static Switches read_switches() {
    Switches w;
    w.pdl = env_int("POLESTAR_PDL", w.pdl);
    w.evict_first = env_int("POLESTAR_GEMM_EVICT_FIRST", w.evict_first);
    w.fuse_select = env_int("POLESTAR_FUSE_SELECT", w.fuse_select);
    w.chain = env_int("POLESTAR_CHAIN", w.chain);
    w.stages = env_int("POLESTAR_GEMM_STAGES", w.stages);
    w.pair_rows = env_int("POLESTAR_GEMM_PAIR_ROWS", w.pair_rows);
    w.epi_groups = env_int("POLESTAR_GEMM_EPI_GROUPS", w.epi_groups);
    w.align_pct = env_int("POLESTAR_GEMM_ALIGN_PCT", w.align_pct);
    w.half_align = env_int("POLESTAR_GEMM_HALF_ALIGN", w.half_align);
    w.attn_kernel = env_int("POLESTAR_ATTN_KERNEL", w.attn_kernel);
    w.attn_simt = env_int("POLESTAR_ATTN_SIMT", w.attn_simt);
    w.refresh_simt = env_int("POLESTAR_REFRESH_SIMT", w.refresh_simt);
    w.fuse_prep = env_int("POLESTAR_FUSE_PREP", w.fuse_prep);
    w.fold_norm = env_int("POLESTAR_FOLD_NORM", w.fold_norm);
    w.accumulate = env_int("POLESTAR_GEMM_ACCUMULATE", w.accumulate);
    w.one_tall = env_int("POLESTAR_GEMM_ONE_TALL", w.one_tall);
    w.tall_rows = env_int("POLESTAR_GEMM_TALL_ROWS", w.tall_rows);
    w.tall_rows_ffn = env_int("POLESTAR_GEMM_TALL_ROWS_FFN", getenv("POLESTAR_GEMM_TALL_ROWS") ? w.tall_rows : w.tall_rows_ffn);
    w.chain_qkv = env_int("POLESTAR_CHAIN_QKV", w.chain_qkv);
    w.l2promo = env_int("POLESTAR_TMA_L2PROMO", w.l2promo);
    w.gemm_trace = env_int("POLESTAR_GEMM_TRACE", w.gemm_trace);
    w.kernel_trace = env_int("POLESTAR_KERNEL_TRACE", w.kernel_trace);
    return w;
}
static std::mutex g_mu;                 // guards g_sw and g_dev
static Switches g_sw;                   // switches of the stand-alone kernel calls
static bool g_sw_loaded = false;
static Switches stand_alone_switches() {
    std::lock_guard<std::mutex> lk(g_mu);
    if (!g_sw_loaded) { g_sw = read_switches(); g_sw_loaded = true; }
    return g_sw;
}

// ------------------------------------------------------------------------------------------
// per-device facts: SM count, dynamic shared-memory attributes of the kernels, built-in scratch
// ------------------------------------------------------------------------------------------
struct DevInfo { bool ready = false; int sm_count = 0; int gemm_pairs = 0; };
static const int MAX_DEVICES = 64;
static DevInfo g_dev[MAX_DEVICES];
static int g_last_sm_count = 0;

static cudaError_t set_kernel_attributes();
static int resident_gemm_pairs();
// Facts of the CURRENT device; the first call on a device queries it and raises the shared-memory limits of
// every kernel that needs more than the default there (function attributes are per device).
static int device_info(DevInfo* out) {
    int dev = 0;
    CK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= MAX_DEVICES) return POLESTAR_E_INVAL;
    std::lock_guard<std::mutex> lk(g_mu);
    DevInfo& di = g_dev[dev];
    if (!di.ready) {
        CK(cudaDeviceGetAttribute(&di.sm_count, cudaDevAttrMultiProcessorCount, dev));
        CK(set_kernel_attributes());
        di.gemm_pairs = resident_gemm_pairs();
        di.ready = true;
    }
    g_last_sm_count = di.sm_count;
    *out = di;
    return POLESTAR_OK;
}

// ------------------------------------------------------------------------------------------
// tensor maps (TMA descriptors) through the driver entry point, no libcuda link dependency
// ------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn get_encode_fn() {
    static std::atomic<EncodeTiledFn> fn{nullptr};
    EncodeTiledFn f = fn.load();
    if (!f) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess) {
            f = (EncodeTiledFn)p;
            fn.store(f);
        }
    }
    return f;
}
// bf16 matrix [rows, K] row-major, box = box_rows x 64 elements, 128-byte swizzle
static bool make_map(CUtensorMap* out, const void* base, uint64_t rows, uint64_t K, uint32_t box_rows, int l2promo) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {K, rows};
    cuuint64_t strides[1] = {K * 2};
    cuuint32_t box[2] = {64, box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, (CUtensorMapL2promotion)l2promo,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Tensor maps of one context (its weights and staging buffers at the handful of row counts a decode uses);
// owned by the context, so it is bounded by the context's buffers and needs no lock.
// bf16 tensor [batch][rows][width] (row-major), box = 1 x 128 rows x 64 elements, 128-byte swizzle: rows beyond
// `rows` are out of bounds per batch entry and arrive as zeros
static bool make_map3(CUtensorMap* out, const void* base, uint64_t batch, uint64_t rows, uint64_t width, int l2promo) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    cuuint64_t dims[3] = {width, rows, batch};
    cuuint64_t strides[2] = {width * 2, rows * width * 2};
    cuuint32_t box[3] = {64, 128, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    return fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, (CUtensorMapL2promotion)l2promo,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct MapCache {
    std::map<std::tuple<const void*, uint64_t, uint64_t, uint32_t>, CUtensorMap> m;
    int l2promo = (int)CU_TENSOR_MAP_L2_PROMOTION_L2_128B;
    // [batch][rows][width] tensors (K / V caches): keyed with box_rows = 0x80000000 | batch
    const CUtensorMap* get3(const void* base, uint64_t batch, uint64_t rows, uint64_t width) {
        auto key = std::make_tuple(base, rows, width, (uint32_t)(0x80000000u | (uint32_t)batch));
        auto it = m.find(key);
        if (it != m.end()) return &it->second;
        CUtensorMap tm;
        if (!make_map3(&tm, base, batch, rows, width, l2promo)) return nullptr;
        return &m.emplace(key, tm).first->second;
    }
    const CUtensorMap* get(const void* base, uint64_t rows, uint64_t K, uint32_t box_rows) {
        auto key = std::make_tuple(base, rows, K, box_rows);
        auto it = m.find(key);
        if (it != m.end()) return &it->second;
        CUtensorMap tm;
        if (!make_map(&tm, base, rows, K, box_rows, l2promo)) return nullptr;
        return &m.emplace(key, tm).first->second;
    }
};

// ------------------------------------------------------------------------------------------
// GEMM dispatch
// ------------------------------------------------------------------------------------------
struct GemmWs {
    float* partial = nullptr; size_t partial_bytes = 0;
    int* counters = nullptr; int n_counters = 0;
    int* status = nullptr;
    unsigned* post_counter = nullptr;      // grid-wide arrival counter of GEMMs with appended row work (never reset)
    mutable unsigned post_total = 0;       // its value once every launch so far has completed
    unsigned* chain_counter = nullptr;     // the same for chained launches
    mutable unsigned chain_total = 0;
    int sms = 148;                         // SMs of the device the launches go to
    int pairs = 0;                         // CTA pairs (clusters of two) of the pair GEMM that are resident at once; 0: pairs unavailable
    Switches sw;
};

// bf16 matrices with out % 256 == 0 and in % 64 == 0 are stored tile-major (see polestar.h)
static bool weight_is_tiled(int dtype, int n_out, int k) { return dtype == POLESTAR_BF16 && n_out % 256 == 0 && k % 64 == 0; }

template <typename T, int EPI>
static int launch_gemm_simt(const void* A, const void* W, int M, int N_out, int K, const EpiArgs& e, cudaStream_t st) {
    if (M <= 0) return POLESTAR_OK;
    dim3 grid((N_out + 63) / 64, (M + 63) / 64);
    const int w_tiled = weight_is_tiled(sizeof(T) == 2 ? POLESTAR_BF16 : POLESTAR_F32, N_out, K) ? 1 : 0;
    gemm_simt_kernel<T, EPI><<<grid, 256, 0, st>>>((const T*)A, (const T*)W, M, N_out, K, w_tiled, e);
    CK(cudaGetLastError());
    return POLESTAR_OK;
}

// stream-K grid of a GEMM with M rows: G CTAs over U units
static void sk_grid(const GemmWs& ws, int M, int N_out, int K, long long* U, long long* G, int BT = tc::BLOCK_T, int units = 0) {
    const int tiles_f = N_out / tc::BLOCK_F, tiles_t = (M + BT - 1) / BT;
    const int sms = units > 0 ? units : ws.sms;           // scheduling units: SMs, or resident CTA pairs
    *U = (long long)tiles_f * tiles_t * (K / 64);
    long long g = std::min<long long>((long long)sms, *U);
    const long long tiles = (long long)tiles_f * tiles_t;
    const long long mult = (g / tiles) * tiles;
    const int pct = ws.sw.align_pct;
    if (mult > 0 && mult * 100 >= (long long)sms * pct) g = mult;
    else if (tiles % 2 == 0 && ws.sw.half_align) {
        // next best: a multiple of half the tile count, so that CTA ranges cross a tile boundary only in every
        // third (fifth, ...) CTA instead of in nearly all of them
        const long long half = tiles / 2, mult2 = (g / half) * half;
        if (mult2 > 0 && mult2 * 100 >= (long long)sms * pct) g = mult2;
    }
    *G = g;
}

template <int EPI>
static int launch_gemm_tc(MapCache& maps, const GemmWs& ws, const void* A, const void* W, int M,
                          int N_out, int K, const EpiArgs& e, cudaStream_t st,
                          const PostArgs* post = nullptr, const tc::SelFuse* sel = nullptr) {
    if (M <= 0) return POLESTAR_OK;
    // weights: tile-major [chunks * 256][64]; activations: exactly M rows, so that the rows of a token tile
    // beyond M are out of bounds and arrive as zeros without being read
    // Steps of several hundred rows (operands from L2, tensor-bound): CTA tiles of 256 tokens, two MMAs per k step on
    // one weight tile (64 KB of operands per k block for twice the work of 48 KB)
    // From POLESTAR_GEMM_PAIR_ROWS rows on: CTA pairs on tiles of 256 tokens (one MMA over both SMs, half a weight tile each)
    const bool pair = ws.pairs > 0 && M >= ws.sw.pair_rows && !(sel && sel->on);
    // (129 - 256 rows, e.g. a refresh step plus its proxy rows: one 256-token tile keeps the step a single token tile, so
    // every weight byte is still read once and streamed with evict_first, instead of two token tiles sharing the weights)
    const bool one_tall = M > tc::BLOCK_T && M <= 2 * tc::BLOCK_T && ws.sw.one_tall;
    const int TT = (!pair && (one_tall || M >= (EPI == EPI_SWIGLU ? ws.sw.tall_rows_ffn : ws.sw.tall_rows))) ? 2 : 1;
    const int BT = tc::BLOCK_T * (pair ? 2 : TT);          // tokens per scheduling unit's tile
    const int tiles_f = N_out / tc::BLOCK_F, tiles_t = (M + BT - 1) / BT;
    // When a multiple of the tile count fits on >= 85 % of the SMs, the grid takes it: CTA ranges then never
    // cross a tile boundary, so every CTA has one segment (one fix-up instead of two, or none at all).
    const CUtensorMap* mw = maps.get(W, (uint64_t)N_out * (uint64_t)(K / 64), 64, pair ? tc::BLOCK_F / 2 : tc::BLOCK_F);
    const CUtensorMap* ma = maps.get(A, (uint64_t)M, (uint64_t)K, tc::BLOCK_T);
    if (!mw || !ma) return POLESTAR_E_CUDA;
    long long U, G;
    if (pair) {
        // the pair is the scheduling unit: G counts pairs here, the launch has twice as many CTAs
        sk_grid(ws, M, N_out, K, &U, &G, BT, ws.pairs);
        while (G > 1 && ((size_t)4 * G * tc::BLOCK_T * tc::BLOCK_F * 4 + 16384 + 65536 > ws.partial_bytes)) --G;
        if (2 * tiles_f * tiles_t + 2 > ws.n_counters / 2) return POLESTAR_E_INVAL;
    } else {
        sk_grid(ws, M, N_out, K, &U, &G, BT, ws.sms);
        while (G > 1 && ((size_t)2 * G * BT * tc::BLOCK_F * 4 + 16384 + 65536 > ws.partial_bytes)) --G;
        if (tiles_f * tiles_t > ws.n_counters / 2) return POLESTAR_E_INVAL;
    }
    tc::SkArgs g;
    g.M = M; g.N_out = N_out; g.K = K; g.tiles_f = tiles_f; g.tiles_t = tiles_t;
    // Three stages (145 KB) for the weight-bound steps: measured +2 % tokens/s over four (the HBM stream needs no more in
    // flight, and less shared memory per block leaves room for the next kernel's blocks to become resident early); two
    // stages are 4 % slower.  Four stages when operands come from L2 (several token tiles).
    g.stages = std::max(2, std::min(4, ws.sw.stages > 0 ? ws.sw.stages : (tiles_t == 1 ? 3 : 4)));
    if (TT == 2) g.stages = std::min(g.stages, 3);          // 64 KB per stage
    if (pair) g.stages = 6;                                 // 32 KB per stage and CTA
    g.partial = ws.partial; g.tile_counter = ws.counters; g.done_offset = ws.n_counters / 2; g.status = ws.status;
    g.w_stream = (g.tiles_t == 1 && ws.sw.evict_first) ? 1 : 0;
    g.epi_groups = g.tiles_t > 1 ? std::max(1, std::min(3, ws.sw.epi_groups)) : 1;
    // POLESTAR_TRACE builds: nanosecond stamps of the launches of one epilogue kind, kept in the tail of the partial workspace
    g.trace = (ws.sw.gemm_trace == EPI) ? (long long*)((char*)ws.partial + ws.partial_bytes - 16384) : nullptr;
    const size_t smem = pair ? (size_t)g.stages * (tc::A_BYTES + tc::W_BYTES / 2) + 1024
                             : (size_t)g.stages * (tc::STAGE_BYTES + (TT - 1) * tc::A_BYTES) + 1024;
    auto kern = TT == 2 ? tc::gemm_sk_kernel<__nv_bfloat16, EPI, 2> : tc::gemm_sk_kernel<__nv_bfloat16, EPI, 1>;
    const unsigned n_ctas = (unsigned)(pair ? 2 * G : G);
    PostArgs pa;
    memset(&pa, 0, sizeof(pa));
    if (post && post->kind && ws.post_counter) {
        pa = *post;
        pa.counter = ws.post_counter;
        ws.post_total += n_ctas;
        pa.expect = ws.post_total;
    }
    tc::SelFuse sfz;
    if (sel) sfz = *sel; else memset(&sfz, 0, sizeof(sfz));
    if (sfz.on) g.epi_groups = 1;          // the selection runs on warps 6-13 of the first CTA
    if (pair) {
        CK(launch_k_cluster(tc::gemm_sk_kernel<__nv_bfloat16, EPI, 1, 2>, dim3(n_ctas), dim3(tc::FIX_THREADS), smem, st, 2u, *mw, *ma, g, e, pa, sfz));
        return POLESTAR_OK;
    }
    CK(launch_k(kern, dim3((unsigned)G), dim3(tc::FIX_THREADS), smem, st, *mw, *ma, g, e, pa, sfz));
    return POLESTAR_OK;
}

// Block size of the row-wise staging kernels (one CTA per row, the row in registers): 512 threads for the few rows of a
// decoding step (latency: every thread has one or two 16-byte loads in flight), 128 threads when a step has hundreds of
// rows, so that several rows share an SM instead of queueing one 512-thread CTA after the other.
static int norm_threads(int rows, int d) {
    return (rows >= 256 && d <= 4 * NORM_VPT * 128) ? 128 : NORM_THREADS;
}

// Attention + drift on tensor cores (attn_tc.cuh): bf16, head_dim 128, at most atc::MAX_N keys.
static bool attention_tc_applies(const AttnArgs& a) {
    return a.head_dim == atc::DH && a.N <= atc::MAX_N && a.N > 0 && (a.n_heads * a.head_dim) % 64 == 0 &&
           (a.n_kv * a.head_dim) % 64 == 0;
}
static int launch_attention_tc(MapCache& maps, const AttnArgs& a, cudaStream_t st, int* status) {
    if (a.n_rows <= 0) return POLESTAR_OK;
    atc::Args g;
    memset(&g, 0, sizeof(g));
    g.a = a;
    const int batch = a.batch > 0 ? a.batch : 1;
    g.rows_per_seq = a.rows_per_seq > 0 ? a.rows_per_seq : a.n_rows;
    g.tiles_per_seq = (g.rows_per_seq + atc::ROWS - 1) / atc::ROWS;
    const int tiles_k = (a.N + atc::KEYS - 1) / atc::KEYS;
    g.kt = tiles_k > atc::MAX_CL ? 2 : 1;
    g.cl = (tiles_k + g.kt - 1) / g.kt;
    g.status = status;
    const int dq = a.n_heads * a.head_dim, dkv = a.n_kv * a.head_dim;
    const int kv_batch = a.rows ? batch : 1;
    const CUtensorMap* mq = maps.get(a.q, (uint64_t)a.n_rows, (uint64_t)dq, atc::ROWS);
    const CUtensorMap* mk = maps.get3(a.kc, (uint64_t)kv_batch, (uint64_t)a.N, (uint64_t)dkv);
    const CUtensorMap* mv = maps.get3(a.vc, (uint64_t)kv_batch, (uint64_t)a.N, (uint64_t)dkv);
    if (!mq || !mk || !mv) return POLESTAR_E_CUDA;
    dim3 grid((unsigned)(g.cl * g.tiles_per_seq * batch), (unsigned)a.n_heads);
    const size_t smem = atc::smem_bytes(g.kt);
    // (always a cluster launch, also for a single key range: the kernel addresses its own CTA through the cluster window)
    CK(launch_k_cluster(atc::attention_tc_kernel, grid, dim3(atc::THREADS), smem, st, (unsigned)g.cl, *mq, *mk, *mv, g));
    return POLESTAR_OK;
}

// The streaming form (attn_stream.cuh): one CTA per (128 rows, head) walks all key tiles; any number of keys.
static bool attention_stream_applies(const AttnArgs& a) {
    return a.head_dim == ast::DH && a.N > 0 && (a.n_heads * a.head_dim) % 64 == 0 && (a.n_kv * a.head_dim) % 64 == 0;
}
// Which of the two tensor-core kernels: the streaming one as soon as its grid (row tiles x heads x sequences) fills a
// good part of the GPU -- block entries, batches, long sequences (measured: 512 x 512 keys 43 us against 80 us,
// 2048 x 2048 keys 0.6 ms against 1.4 ms) -- or the keys exceed what a cluster of key ranges covers; the cluster
// kernel for the small steps of one short sequence, where spreading the keys over SMs wins (128 x 512: 20 us against 37 us).
static bool attention_prefers_stream(const AttnArgs& a) {
    const int batch = a.batch > 0 ? a.batch : 1;
    const int rps = a.rows_per_seq > 0 ? a.rows_per_seq : a.n_rows;
    const long long ctas = (long long)((rps + ast::ROWS - 1) / ast::ROWS) * batch * a.n_heads;
    return ctas >= 64 || a.N > atc::MAX_N;
}
static int launch_attention_stream(MapCache& maps, const AttnArgs& a, cudaStream_t st, int* status) {
    if (a.n_rows <= 0) return POLESTAR_OK;
    ast::Args g;
    memset(&g, 0, sizeof(g));
    g.a = a;
    const int batch = a.batch > 0 ? a.batch : 1;
    g.rows_per_seq = a.rows_per_seq > 0 ? a.rows_per_seq : a.n_rows;
    g.tiles_per_seq = (g.rows_per_seq + ast::ROWS - 1) / ast::ROWS;
    g.status = status;
    const int dq = a.n_heads * a.head_dim, dkv = a.n_kv * a.head_dim;
    const int kv_batch = a.rows ? batch : 1;
    const CUtensorMap* mq = maps.get(a.q, (uint64_t)a.n_rows, (uint64_t)dq, ast::ROWS);
    const CUtensorMap* mk = maps.get3(a.kc, (uint64_t)kv_batch, (uint64_t)a.N, (uint64_t)dkv);
    const CUtensorMap* mv = maps.get3(a.vc, (uint64_t)kv_batch, (uint64_t)a.N, (uint64_t)dkv);
    if (!mq || !mk || !mv) return POLESTAR_E_CUDA;
    dim3 grid((unsigned)(g.tiles_per_seq * batch), (unsigned)a.n_heads);
    CK(launch_k(ast::attention_stream_kernel, grid, dim3(ast::THREADS), ast::smem_bytes(), st, *mq, *mk, *mv, g));
    return POLESTAR_OK;
}

// ------------------------------------------------------------------------------------------
// context
// ------------------------------------------------------------------------------------------
struct Plan {
    size_t total = 0;
    size_t take(size_t bytes) {
        const size_t o = total;
        total += (bytes + 1023) & ~(size_t)1023;
        return o;
    }
};

struct Buffers {
    // persistent
    int* y; float2* rope; char* kc; char* vc; float* hc; float* pprev; float* aprev; float* pprev_lse; float* aprev_lse;
    float* theta; int* theta_cnt;
    int* tok_at_h0; float* drift; int* sel_idx; int* sel_cnt; unsigned char* patch; int* forced_idx; int* forced_cnt;
    int* forced_commit; int* forced_tok; float* conf; int* yhat; float* delta; float* Delta; float* taud; int* commit_flags;
    int* own_flags; int* suffix_flags; int* seq_info; int* head_count; int* suf_seq; int* suf_w; int* stats; int* status;
    int* list_count; float* hidden_keep;
    int* labels; int* zpos; int* zcnt; int* members; int* moff; int* forced_labels; float* zbuf; float* kcent;   // centroid proxies
    unsigned char* hq; unsigned char* hs; float* z0;                                                             // NVFP4 residual cache
    unsigned char* fmask; unsigned char* fq; unsigned char* fs;                                                  // imposed codes (checking only)
    // scratch
    Row* rows; unsigned char* kvflag; float* x; float* x1; float* packet; char* a_buf; char* q_buf; char* o_buf;
    char* g_buf; float* kl; int* list; long long* fold_ss; HeadSrc* head_list; char* a_head; float* logits; ConfPart* conf_part;
    float* gemm_partial; int* gemm_counters;
};

static const int CONF_CHUNKS = 32;
static const int FORCED_COMMIT_MAX = 512;
static const size_t GEMM_PARTIAL_BYTES = ((size_t)80 << 20) + 16384 + 65536;   // 2 slots x 148 CTAs x 256 x 256 fp32
// One projection of a chained launch (gemm_chain.cuh): A [M, K] x W [N_out, K]^T with epilogue `epi`.
struct ChainSpec {
    const void* A; const void* W;
    int N_out, K, epi, norm_after;
    EpiArgs e;
    PostArgs post;
};
// Launches the projections as one persistent kernel when the chain applies (M <= 128 rows, tile-major weights);
// otherwise *applies = false and nothing is launched.
template <typename T>
static int launch_gemm_chain(MapCache& maps, const GemmWs& ws, const ChainSpec* sp, int n, int M, cudaStream_t st,
                             const tc::SelFuse* sel, bool* applies) {
    *applies = false;
    if (n < 2 || n > tc::CHAIN_MAX || M <= 0 || M > tc::BLOCK_T || !ws.chain_counter) return POLESTAR_OK;
    long long G0 = 0, Gp[tc::CHAIN_MAX];
    for (int i = 0; i < n; ++i) {
        if (sp[i].N_out % tc::BLOCK_F || sp[i].K % 64) return POLESTAR_OK;
        long long U;
        sk_grid(ws, M, sp[i].N_out, sp[i].K, &U, &Gp[i]);
        if (sp[i].N_out / tc::BLOCK_F > Gp[i]) return POLESTAR_OK;
        G0 = std::max(G0, Gp[i]);
    }
    if ((size_t)2 * G0 * tc::BLOCK_T * tc::BLOCK_F * 4 + 16384 + 65536 > ws.partial_bytes) return POLESTAR_OK;
    tc::ChainMaps cm;
    tc::ChainArgs ca;
    memset(&ca, 0, sizeof(ca));
    int n_bar = 0;
    for (int i = 0; i < n; ++i) {
        const CUtensorMap* mw = maps.get(sp[i].W, (uint64_t)sp[i].N_out * (uint64_t)(sp[i].K / 64), 64, tc::BLOCK_F);
        const CUtensorMap* ma = maps.get(sp[i].A, (uint64_t)M, (uint64_t)sp[i].K, tc::BLOCK_T);
        if (!mw || !ma) return POLESTAR_E_CUDA;
        cm.w[i] = *mw; cm.a[i] = *ma;
        tc::ChainProb& P = ca.p[i];
        P.M = M; P.N_out = sp[i].N_out; P.K = sp[i].K; P.tiles_f = sp[i].N_out / tc::BLOCK_F; P.G = (int)Gp[i];
        P.epi = sp[i].epi; P.norm_after = (i + 1 < n) ? sp[i].norm_after : 0;      // 0 none, 1 RMSNorm rows, 2 QKV input staging
        P.e = sp[i].e; P.post = sp[i].post;
        if (i + 1 < n) n_bar += 1 + (P.norm_after ? 1 : 0);
    }
    for (int i = n; i < tc::CHAIN_MAX; ++i) { cm.w[i] = cm.w[0]; cm.a[i] = cm.a[0]; }
    ca.n = n;
    ca.stages = std::max(2, std::min(4, ws.sw.stages > 0 ? ws.sw.stages : 3));
    ca.partial = ws.partial; ca.tile_counter = ws.counters; ca.done_offset = ws.n_counters / 2; ca.status = ws.status;
    ca.bar_counter = ws.chain_counter;
    ca.bar_base = ws.chain_total;
    ws.chain_total += (unsigned)(n_bar * G0);
    tc::SelFuse sfz;
    if (sel) sfz = *sel; else memset(&sfz, 0, sizeof(sfz));
    const size_t smem = (size_t)ca.stages * tc::STAGE_BYTES + 1024;
    CK(launch_k(tc::gemm_chain_kernel<T>, dim3((unsigned)G0), dim3(tc::FIX_THREADS), smem, st, cm, ca, sfz));
    *applies = true;
    return POLESTAR_OK;
}

static const int GEMM_COUNTERS = 1 << 17;     // arrivals + finished shares for up to 65536 output tiles

struct polestar_ctx {
    polestar_model m;
    polestar_params p;
    std::vector<const void*> wqkv, wo, wgu, wd;
    std::vector<const float*> n1, n2;
    const void *embed, *lm_head;
    const float* final_norm;
    cudaStream_t st;
    char* ws;
    Buffers b;
    MapCache maps;
    GemmWs gws;
    int es;          // element size of the model dtype
    int device = 0;  // CUDA device the context was created on
    int sms = 148;
    Switches sw;
    int N, B, W_max, n_blocks, M_max, rows_lm;
    // controller
    int block = 0;
    bool need_entry = true, pending = false, done = false;
    bool trace_installed = false;
    bool failed = false;     // a device-side wait timed out: counters and caches are in an unknown state
    int steps_used = 0;
    long long forwards = 0, generated = 0, generated_non_eos = 0;
    std::vector<int> cum;
    StepDesc last_sd;
    int last_act_row_off = 0;
    bool forced_select = false, forced_commit = false, forced_tokens = false, forced_labels = false, forced_codes = false;
    int forced_commit_n = 0;
    int* seq_info_host = nullptr;          // pinned: bs * 8 + 8 words
    // launch accounting and optional per-family device timing (POLESTAR_FLAG_PROFILE)
    long long launches = 0;
    struct ProfRec { int fam; size_t ev; double bytes, flops; };
    std::vector<cudaEvent_t> prof_ev;
    std::vector<ProfRec> prof_recs;
    size_t prof_used = 0;
    double prof_acc[POLESTAR_PROF_FAMILIES][4] = {};
};

// Scope of one kernel family inside a forward: counts launches, and with FLAG_PROFILE brackets the
// launches with CUDA events that polestar_commit turns into per-family device times.
struct Scope {
    polestar_ctx* c;
    bool on;
    size_t ev = 0;
    Scope(polestar_ctx* c_, int fam, double bytes, double flops, int n_launches) : c(c_) {
        c->launches += n_launches;
        on = (c->p.flags & POLESTAR_FLAG_PROFILE) != 0;
        if (!on) return;
        while (c->prof_ev.size() < c->prof_used + 2) {
            cudaEvent_t e;
            if (cudaEventCreate(&e) != cudaSuccess) { on = false; return; }
            c->prof_ev.push_back(e);
        }
        ev = c->prof_used;
        c->prof_used += 2;
        cudaEventRecord(c->prof_ev[ev], c->st);
        c->prof_recs.push_back({fam, ev, bytes, flops});
    }
    ~Scope() {
        if (on) cudaEventRecord(c->prof_ev[ev + 1], c->st);
    }
};

static bool valid_cfg(const polestar_model* m, const polestar_params* p) {
    if (!m || !p) return false;
    if (m->n_layers <= 0 || m->d_model <= 0 || m->n_heads <= 0 || m->n_kv_heads <= 0 || m->head_dim <= 0) return false;
    if (m->n_heads % m->n_kv_heads) return false;
    if (m->head_dim % 2 || m->head_dim > 256 || m->d_ffn <= 0 || m->vocab < 4 || m->vocab % 2) return false;
    if (m->dtype != POLESTAR_F32 && m->dtype != POLESTAR_BF16) return false;
    if (m->mask_id < 0 || m->mask_id >= m->vocab || m->eos_id < 0 || m->eos_id >= m->vocab) return false;
    if (m->d_model % 8 || (m->n_heads * m->head_dim) % 8 || m->d_ffn % 8) return false;
    if (m->d_model > 4 * NORM_VPT * NORM_THREADS) return false;
    if (p->batch <= 0 || p->batch > POLESTAR_MAX_BATCH) return false;
    if (p->prompt_len < 0 || p->gen_len <= 0 || p->block <= 0 || p->block > 256) return false;
    if (p->gen_len % p->block) return false;
    if (p->max_steps <= 0 || p->win_prefix_blocks < 0 || p->win_suffix_blocks < 0 || p->full_entry_period <= 0) return false;
    if (p->select_mode < 0 || p->select_mode > POLESTAR_SELECT_CLUSTER_TOPK || p->hist < 0 || p->hist > 64) return false;
    const long long N = (long long)p->prompt_len + p->gen_len;
    if (N > 65536) return false;
    const long long wmax = std::min<long long>((long long)(p->win_prefix_blocks + p->win_suffix_blocks) * p->block, N - p->block);
    if (wmax > 1024) return false;
    if (p->select_mode == POLESTAR_SELECT_CLUSTER_TOPK) {
        // proxies ride behind the window rows; their drift shares the window's drift row; selection by rank counting
        if (p->n_clusters < 1 || p->n_clusters > KM_MAX_K || p->cluster_k < 0 || p->kmeans_iters < 1 || p->kmeans_iters > 16) return false;
        if (wmax > SEL_SMALL_W || p->n_clusters > std::max<long long>(wmax, 1) || m->d_model % 4) return false;
    }
    if (p->flags & POLESTAR_FLAG_NVFP4_HCACHE) {
        // residuals are taken against cluster centroids; whole warps work on a row's 16-channel groups
        if (p->select_mode != POLESTAR_SELECT_CLUSTER_TOPK || (p->flags & POLESTAR_FLAG_NOCACHE) || m->d_model % 128) return false;
    }
    return true;
}

// proxy rows per sequence (the full-recompute baseline has no cache to calibrate, hence no proxies)
static int n_proxies(const polestar_params* p) {
    return (p->select_mode == POLESTAR_SELECT_CLUSTER_TOPK && !(p->flags & POLESTAR_FLAG_NOCACHE)) ? p->n_clusters : 0;
}

static int window_max(const polestar_params* p) {
    const long long N = (long long)p->prompt_len + p->gen_len;
    long long w = std::min<long long>((long long)(p->win_prefix_blocks + p->win_suffix_blocks) * p->block, N - p->block);
    return (int)std::max<long long>(w, 1);
}

static size_t make_plan(const polestar_model* m, const polestar_params* p, Buffers* b, char* base) {
    Plan pl;
    const size_t es = m->dtype == POLESTAR_BF16 ? 2 : 4;
    const size_t L = m->n_layers, bs = p->batch, N = (size_t)p->prompt_len + p->gen_len, B = p->block;
    const size_t d = m->d_model, dq = (size_t)m->n_heads * m->head_dim, dkv = (size_t)m->n_kv_heads * m->head_dim;
    const size_t F = m->d_ffn, V = m->vocab, nh = m->n_heads;
    const size_t Wm = window_max(p);
    const size_t n_suf = std::min<size_t>((size_t)p->win_suffix_blocks * B, Wm);
    const size_t Kp = n_proxies(p);                    // proxy rows per sequence (centroid proxies)
    const size_t rec = Kp ? Kp : Wm;                   // recorded drift rows per sequence and layer
    const size_t Mmax = bs * (std::max(N, B + Wm) + Kp);
    const size_t rows_lm = bs * (B + n_suf);
#define TAKE(field, type, count)                                  \
    do {                                                          \
        const size_t _o = pl.take((size_t)(count) * sizeof(type)); \
        if (b) b->field = (type*)(base + _o);                     \
    } while (0)
    TAKE(y, int, bs * N);
    TAKE(rope, float2, N * (m->head_dim / 2));
    TAKE(kc, char, L * bs * N * dkv * es);
    TAKE(vc, char, L * bs * N * dkv * es);
    const bool quant = (p->flags & POLESTAR_FLAG_NVFP4_HCACHE) != 0;
    TAKE(hc, float, quant ? 1 : L * bs * Wm * d);
    TAKE(pprev, float, L * bs * rec * nh * N);
    TAKE(aprev, float, bs * B * nh * N);
    TAKE(pprev_lse, float, L * bs * rec * nh);
    TAKE(aprev_lse, float, bs * B * nh);
    TAKE(theta, float, bs * std::max<size_t>(1, p->hist) * B);
    TAKE(theta_cnt, int, bs);
    TAKE(tok_at_h0, int, bs * Wm);
    TAKE(drift, float, L * bs * Wm);
    TAKE(sel_idx, int, L * bs * Wm);
    TAKE(sel_cnt, int, L * bs);
    TAKE(patch, unsigned char, (L + 1) * bs * Wm);
    TAKE(forced_idx, int, L * bs * Wm);
    TAKE(forced_cnt, int, L * bs);
    TAKE(forced_commit, int, bs * FORCED_COMMIT_MAX);
    TAKE(forced_tok, int, bs * FORCED_COMMIT_MAX);
    TAKE(conf, float, rows_lm);
    TAKE(yhat, int, rows_lm);
    TAKE(delta, float, bs * B);
    TAKE(Delta, float, bs * B);
    TAKE(taud, float, bs * B);
    TAKE(commit_flags, int, bs * B);
    TAKE(own_flags, int, bs * B);
    TAKE(suffix_flags, int, bs * Wm);
    TAKE(seq_info, int, bs * 8 + 8);
    TAKE(head_count, int, 1);
    TAKE(suf_seq, int, bs * Wm);
    TAKE(suf_w, int, bs * Wm);
    TAKE(stats, int, 4);
    TAKE(status, int, 1);
    TAKE(list_count, int, 1);
    TAKE(hidden_keep, float, (p->flags & POLESTAR_FLAG_KEEP_HIDDEN) ? (L + 1) * bs * B * d : 1);
    TAKE(labels, int, Kp ? L * bs * Wm : 1);
    TAKE(zpos, int, Kp ? L * bs * Kp : 1);
    TAKE(zcnt, int, Kp ? L * bs * Kp : 1);
    TAKE(members, int, Kp ? L * bs * Wm : 1);
    TAKE(moff, int, Kp ? L * bs * (Kp + 1) : 1);
    TAKE(forced_labels, int, Kp ? L * bs * Wm : 1);
    TAKE(zbuf, float, Kp ? bs * Kp * d : 1);
    TAKE(kcent, float, Kp ? bs * (Kp * d + Wm) : 1);
    TAKE(hq, unsigned char, quant ? L * bs * Wm * (d / 2) : 1);
    TAKE(hs, unsigned char, quant ? L * bs * Wm * (d / 16) : 1);
    TAKE(z0, float, quant ? L * bs * Kp * d : 1);
    const bool imposed = quant && (p->flags & POLESTAR_FLAG_KEEP_HIDDEN);
    TAKE(fmask, unsigned char, imposed ? L * bs * Wm : 1);
    TAKE(fq, unsigned char, imposed ? L * bs * Wm * (d / 2) : 1);
    TAKE(fs, unsigned char, imposed ? L * bs * Wm * (d / 16) : 1);
    TAKE(rows, Row, Mmax);
    TAKE(kvflag, unsigned char, Mmax);
    TAKE(x, float, Mmax * d);
    TAKE(x1, float, Mmax * d);
    TAKE(packet, float, bs * Wm * d);
    TAKE(a_buf, char, Mmax * d * es);
    TAKE(q_buf, char, Mmax * dq * es);
    TAKE(o_buf, char, Mmax * dq * es);
    TAKE(g_buf, char, Mmax * F * es);
    TAKE(kl, float, Mmax * nh);
    TAKE(list, int, Mmax);
    TAKE(fold_ss, long long, (size_t)2 * L * Mmax);
    TAKE(head_list, HeadSrc, rows_lm);
    TAKE(a_head, char, rows_lm * d * es);
    TAKE(logits, float, rows_lm * V);
    TAKE(conf_part, ConfPart, rows_lm * CONF_CHUNKS);
    TAKE(gemm_partial, float, GEMM_PARTIAL_BYTES / 4);
    TAKE(gemm_counters, int, GEMM_COUNTERS);
#undef TAKE
    return pl.total;
}

extern "C" size_t polestar_workspace_bytes(const polestar_model* m, const polestar_params* p) {
    if (!valid_cfg(m, p)) return 0;
    // the plan is laid out from a 1024-byte boundary inside the caller's buffer: a 256-byte aligned base can lose 768 bytes
    return make_plan(m, p, nullptr, nullptr) + 1024;
}

extern "C" int polestar_sm_count(void) {
    std::lock_guard<std::mutex> lk(g_mu);
    return g_last_sm_count;
}

extern "C" int polestar_reload_env(void) {
    std::lock_guard<std::mutex> lk(g_mu);
    g_sw = read_switches();
    g_sw_loaded = true;
    g_use_pdl = g_sw.pdl != 0;
    return POLESTAR_OK;
}

extern "C" const char* polestar_strerror(int code) {
    switch (code) {
        case POLESTAR_OK: return "ok";
        case POLESTAR_E_INVAL: return "invalid argument or unsupported shape";
        case POLESTAR_E_STATE: return "call order violated";
        case POLESTAR_E_NOSPACE: return "workspace too small";
        case POLESTAR_E_CUDA: return cudaGetErrorString(last_cuda_error);
        case POLESTAR_E_NONFINITE: return "non-finite confidence";
        case POLESTAR_E_TIMEOUT: return "device-side wait timed out";
        case POLESTAR_E_DONE: return "decoding already finished";
        default: return "unknown error";
    }
}

static const size_t SIMT_ATTN_SMEM_MAX = 200 * 1024;
// How many clusters of two CTAs of the pair GEMM the device holds at once (its grid-wide counters need every CTA resident)
static int resident_gemm_pairs() {
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3(2 * 148); cfg.blockDim = dim3(tc::FIX_THREADS);
    cfg.dynamicSmemBytes = 6 * (tc::A_BYTES + tc::W_BYTES / 2) + 1024;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    cfg.attrs = at; cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, tc::gemm_sk_kernel<__nv_bfloat16, EPI_QKV, 1, 2>, &cfg) != cudaSuccess) { cudaGetLastError(); return 0; }
    return n;
}

static cudaError_t set_kernel_attributes() {
    cudaError_t e;
    const int gemm_smem = 4 * (int)tc::STAGE_BYTES + 1024;    // four stages of 48 KB + alignment slack
#define PS_ATTR(kern, bytes) if ((e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes)) != cudaSuccess) return e
    PS_ATTR((tc::gemm_sk_kernel<__nv_bfloat16, EPI_QKV>), gemm_smem);
    PS_ATTR((tc::gemm_sk_kernel<__nv_bfloat16, EPI_RESID>), gemm_smem);
    PS_ATTR((tc::gemm_sk_kernel<__nv_bfloat16, EPI_SWIGLU>), gemm_smem);
    PS_ATTR((tc::gemm_sk_kernel<__nv_bfloat16, EPI_DOWN>), gemm_smem);
    PS_ATTR((tc::gemm_sk_kernel<__nv_bfloat16, EPI_LOGITS>), gemm_smem);
    PS_ATTR((tc::gemm_sk_kernel<__nv_bfloat16, EPI_QKV_REFRESH>), gemm_smem);
    PS_ATTR((tc::gemm_sk_kernel<__nv_bfloat16, EPI_QKV, 1, 2>), gemm_smem);
    PS_ATTR((tc::gemm_sk_kernel<__nv_bfloat16, EPI_RESID, 1, 2>), gemm_smem);
    PS_ATTR((tc::gemm_sk_kernel<__nv_bfloat16, EPI_SWIGLU, 1, 2>), gemm_smem);
    PS_ATTR((tc::gemm_sk_kernel<__nv_bfloat16, EPI_DOWN, 1, 2>), gemm_smem);
    PS_ATTR((tc::gemm_sk_kernel<__nv_bfloat16, EPI_LOGITS, 1, 2>), gemm_smem);
    PS_ATTR((tc::gemm_sk_kernel<__nv_bfloat16, EPI_QKV_REFRESH, 1, 2>), gemm_smem);
    PS_ATTR((tc::gemm_sk_kernel<__nv_bfloat16, EPI_QKV, 2>), gemm_smem);
    PS_ATTR((tc::gemm_sk_kernel<__nv_bfloat16, EPI_RESID, 2>), gemm_smem);
    PS_ATTR((tc::gemm_sk_kernel<__nv_bfloat16, EPI_SWIGLU, 2>), gemm_smem);
    PS_ATTR((tc::gemm_sk_kernel<__nv_bfloat16, EPI_DOWN, 2>), gemm_smem);
    PS_ATTR((tc::gemm_sk_kernel<__nv_bfloat16, EPI_LOGITS, 2>), gemm_smem);
    PS_ATTR((tc::gemm_sk_kernel<__nv_bfloat16, EPI_QKV_REFRESH, 2>), gemm_smem);
    PS_ATTR(tc::gemm_chain_kernel<__nv_bfloat16>, gemm_smem);
    PS_ATTR(atc::attention_tc_kernel, (int)atc::smem_bytes(atc::MAX_KT));
    PS_ATTR(kmeans_kernel, KM_SMEM_BYTES);
    PS_ATTR(ast::attention_stream_kernel, (int)ast::smem_bytes());
    PS_ATTR(attention_simt_kernel<float>, (int)SIMT_ATTN_SMEM_MAX);
    PS_ATTR(attention_simt_kernel<__nv_bfloat16>, (int)SIMT_ATTN_SMEM_MAX);
#undef PS_ATTR
    return attention_mma_set_attributes();
}

// ------------------------------------------------------------------------------------------
// one forward
// ------------------------------------------------------------------------------------------
template <typename T>
struct Path {
    static constexpr bool is_bf16 = sizeof(T) == 2;

    template <int EPI>
    static int gemm(polestar_ctx* c, const void* A, const void* W, int M, int N_out, int K,
                    const EpiArgs& e, const PostArgs* post = nullptr, bool* fused = nullptr,
                    const tc::SelFuse* sel = nullptr) {
        if (fused) *fused = false;
        if (is_bf16 && !(c->p.flags & POLESTAR_FLAG_SIMT_GEMM) && K % 64 == 0 && N_out % 256 == 0) {
            const bool fuse = post && post->kind && c->gws.post_counter && post->d <= 4 * NORM_VPT * tc::FIX_THREADS &&
                              c->sw.fuse_prep;      // measured on B200: no faster than the separate kernel
                                                    // (grid-wide counter round trip = kernel boundary)
            if (fused) *fused = fuse;
            return launch_gemm_tc<EPI>(c->maps, c->gws, A, W, M, N_out, K, e, c->st, fuse ? post : nullptr, sel);
        }
        return launch_gemm_simt<T, EPI>(A, W, M, N_out, K, e, c->st);
    }

    static int attention(polestar_ctx* c, const AttnArgs& a) {
        if (is_bf16 && c->m.head_dim == 128 && !c->sw.attn_simt) {
            // one kernel family per context (decided by the shape alone): the families keep stored rows in
            // different forms (scores + log-sum-exp / log-probabilities)
            // Launches that record or compare stored rows all go to the tensor-core kernel.  A launch that touches
            // no stored row (the layers below the last one of a step without refresh) may take either family: for a
            // single block of rows the warp-level kernel's shorter dependency chain wins (11 us against 16 us per
            // layer at the 8B shape), everywhere else the tensor-core kernel does.
            const bool records = a.pprev != nullptr || a.aprev != nullptr;
            // Beyond 1024 keys the warp-level family has a 64-row kernel: it wins where (sequences x heads) fill the GPU (a
            // batch of long sequences, 64 rows each: 85 us against 111 us for the streaming kernel, whose 128-row tiles are half empty).
            const bool fills = (long long)(a.batch > 0 ? a.batch : 1) * a.n_heads >= c->sms;
            const bool few_rows = !records && a.rows_per_seq <= 64 && c->sw.attn_kernel == 0 &&
                                  (a.N <= 1024 || (a.rows_per_seq >= 48 && fills));
            if (attention_stream_applies(a) && !few_rows &&
                (c->sw.attn_kernel == 9 || (c->sw.attn_kernel == 0 && attention_prefers_stream(a))))
                return launch_attention_stream(c->maps, a, c->st, c->b.status);
            if ((c->sw.attn_kernel == 0 || c->sw.attn_kernel == 8) && attention_tc_applies(a) && !few_rows)
                return launch_attention_tc(c->maps, a, c->st, c->b.status);
            if (a.cluster_K > 0 && (a.pprev || a.aprev)) goto simt;      // the warp-level kernels do not know proxy rows
            CK(launch_attention_mma(a, c->st, c->sms, c->sw.attn_kernel));
            return POLESTAR_OK;
        }
    simt:
        const int wpb = 4;
        const size_t smem = (size_t)wpb * a.N * sizeof(float);
        if (smem > SIMT_ATTN_SMEM_MAX) return POLESTAR_E_INVAL;
        dim3 grid((a.n_rows + wpb - 1) / wpb, a.n_heads);
        CK(launch_k(attention_simt_kernel<T>, dim3(grid), dim3(wpb * 32), smem, c->st, a));
        CK(cudaGetLastError());
        return POLESTAR_OK;
    }

    static int forward(polestar_ctx* c, const StepDesc& sd, bool any_refresh) {
        const polestar_model& m = c->m;
        const polestar_params& p = c->p;
        Buffers& b = c->b;
        cudaStream_t st = c->st;
        const int d = m.d_model, dq = m.n_heads * m.head_dim, dkv = m.n_kv_heads * m.head_dim, F = m.d_ffn;
        const int L = m.n_layers, bs = p.batch, N = c->N, B = c->B, Wm = c->W_max;
        const int M = bs * sd.rows_per_seq;
        const int act_off = sd.kind == 2 ? 0 : (sd.act_start - sd.e0);
        const size_t es = sizeof(T);
        const bool within = sd.kind == 2;
        const bool sparse = within && any_refresh;
        int rc;

        const double esd = (double)es;
        const double Mlive = sparse ? (double)bs * (B + std::min(sd.W, (int)(p.select_mode == POLESTAR_SELECT_TOPK_FRAC
                                                       ? floorf(p.select_frac * (float)sd.W + 0.5f)
                                                       : (p.select_mode == POLESTAR_SELECT_TOPK_COUNT ? p.select_k : sd.W))))
                                    : (double)M;
        {
            Scope sc(c, POLESTAR_PROF_STAGE, (double)M * d * (esd + 4), 0, 2);
            CK(launch_k(build_rows_kernel, dim3((M + 255) / 256), dim3(256), 0, st, sd, b.rows));
            CK(cudaMemsetAsync(b.stats, 0, 4 * sizeof(int), st));
            CK(launch_k(embed_rows_kernel<T>, dim3(M), dim3(256), 0, st, sd, b.rows, b.y, (const T*)c->embed, d, b.x, b.packet, b.patch,
                                                   b.tok_at_h0, b.stats));
            CK(cudaGetLastError());
        }

        // Steps whose rows all come straight from the previous projection (within-block steps without refresh): the two
        // RMSNorms of a layer are folded into the projections around them (EpiArgs::fold_*), no staging kernels.
        const bool fold = within && !sparse && is_bf16 && !(p.flags & POLESTAR_FLAG_SIMT_GEMM) && d % 256 == 0 && dq % 64 == 0 &&
                          F % 64 == 0 && (dq + 2 * dkv) % 256 == 0 && (2 * F) % 256 == 0 && c->sw.fold_norm;
        const size_t Mm = (size_t)c->M_max;
        if (fold) CK(cudaMemsetAsync(b.fold_ss, 0, (size_t)2 * L * Mm * sizeof(long long), st));
        bool qkv_staged = false, ffn_staged = false;
        bool qkv_done = false;      // this layer's QKV projection ran at the end of the previous layer's chained kernel
        for (int l = 0; l < L; ++l) {
            char* kc = b.kc + (size_t)l * bs * N * dkv * es;
            char* vc = b.vc + (size_t)l * bs * N * dkv * es;
            float* hc = (p.flags & POLESTAR_FLAG_NVFP4_HCACHE) ? b.hc : b.hc + (size_t)l * bs * Wm * d;     // (unused with the NVFP4 cache)
            float* pprev = b.pprev + (size_t)l * bs * Wm * m.n_heads * N;
            const bool last = l == L - 1;
            // centroid proxies: this layer's cluster tables; at block entry they are made here, from the layer's input rows
            ClusterTabs ct;
            memset(&ct, 0, sizeof(ct));
            const int Kp = sd.K;
            if (Kp > 0) {
                ct.labels = b.labels + (size_t)l * bs * Wm; ct.zpos = b.zpos + (size_t)l * bs * Kp; ct.zcnt = b.zcnt + (size_t)l * bs * Kp;
                ct.members = b.members + (size_t)l * bs * Wm; ct.moff = b.moff + (size_t)l * bs * (Kp + 1); ct.zbuf = b.zbuf; ct.K = Kp;
                if (p.flags & POLESTAR_FLAG_NVFP4_HCACHE) {
                    ct.hq = b.hq + (size_t)l * bs * Wm * (d / 2); ct.hs = b.hs + (size_t)l * bs * Wm * (d / 16);
                    ct.z0 = b.z0 + (size_t)l * bs * Kp * d;
                    if (c->forced_codes) {
                        ct.fmask = b.fmask + (size_t)l * bs * Wm; ct.fq = b.fq + (size_t)l * bs * Wm * (d / 2);
                        ct.fs = b.fs + (size_t)l * bs * Wm * (d / 16);
                    }
                }
                if (!within) {
                    Scope sc(c, POLESTAR_PROF_SELECT, (double)bs * sd.W * d * 4 * 2 * p.kmeans_iters, 0, 1);
                    KmeansArgs ka;
                    memset(&ka, 0, sizeof(ka));
                    ka.x = b.x; ka.d = d; ka.K = Kp; ka.iters = p.kmeans_iters;
                    ka.labels = b.labels + (size_t)l * bs * Wm; ka.zpos = b.zpos + (size_t)l * bs * Kp; ka.zcnt = b.zcnt + (size_t)l * bs * Kp;
                    ka.members = b.members + (size_t)l * bs * Wm; ka.moff = b.moff + (size_t)l * bs * (Kp + 1);
                    ka.forced_labels = b.forced_labels + (size_t)l * bs * Wm; ka.cent = b.kcent; ka.z0 = ct.z0;
                    ka.chunk = std::min((d + 127) & ~127, (KM_SMEM_BYTES / (Kp * 4)) & ~127);
                    CK(launch_k(kmeans_kernel, dim3(KM_CL, bs), dim3(KM_THREADS), (size_t)Kp * ka.chunk * 4, st, sd, ka));
                }
            }
            if (p.flags & POLESTAR_FLAG_KEEP_HIDDEN) {
                Scope sc(c, POLESTAR_PROF_MISC, 0, 0, 1);
                CK(launch_k(keep_hidden_kernel, dim3(bs * B), dim3(256), 0, st, sd, b.x, act_off, d, b.hidden_keep + (size_t)l * bs * B * d));
            }
            if (fold && l > 0) qkv_staged = true;      // the previous down projection stored x * gain and the sums of squares
            if (!qkv_done && !qkv_staged) {      // (else: staged by the previous layer's down projection or chained kernel)
                Scope sc(c, POLESTAR_PROF_STAGE, (double)M * d * (4 + esd), 0, 1);
                CK(launch_k(prep_qkv_kernel<T>, dim3(M), dim3(norm_threads(M, d)), 0, st, sd, b.rows, b.x, hc, b.packet, b.patch + (size_t)l * bs * Wm,
                                                     c->n1[l], m.rms_eps, d, (T*)b.a_buf, b.kvflag, ct));
                CK(cudaGetLastError());
            }
            qkv_staged = false;
            EpiArgs e;
            if (!qkv_done) {
                const double nq = dq + 2 * dkv;
                Scope sc(c, POLESTAR_PROF_GEMM_QKV, (nq * d + (double)M * d + (double)M * nq) * esd, 2.0 * M * nq * d, 1);
                memset(&e, 0, sizeof(e));
                e.rows = b.rows; e.kvflag = b.kvflag; e.rope = b.rope; e.q_out = b.q_buf; e.kc = kc; e.vc = vc;
                e.N_seq = N; e.n_heads = m.n_heads; e.n_kv = m.n_kv_heads; e.head_dim = m.head_dim; e.W_max = Wm;
                e.within = within; e.ld_out = dq;
                e.zpos = ct.zpos; e.n_clusters = Kp;
                if (fold && l > 0) { e.in_ss = b.fold_ss + (size_t)(2 * l) * Mm; e.in_eps = m.rms_eps; e.in_d = d; }
                if ((rc = gemm<EPI_QKV>(c, b.a_buf, c->wqkv[l], M, dq + 2 * dkv, d, e))) return rc;
            }
            qkv_done = false;
            {
                const bool rec_w = sparse || !within;
                const double rec_rows = (rec_w ? (double)bs * (Kp ? Kp : sd.W) : 0.0) + (last ? (double)bs * B : 0.0);
                Scope sc(c, POLESTAR_PROF_ATTENTION,
                         2.0 * bs * N * dkv * esd + 2.0 * M * dq * esd + (sd.record_kl ? 2.0 : 1.0) * rec_rows * m.n_heads * N * 4,
                         4.0 * M * (double)N * dq, 1);
                AttnArgs a;
                memset(&a, 0, sizeof(a));
                a.rows = b.rows; a.n_rows = M; a.q = b.q_buf; a.kc = kc; a.vc = vc; a.out = b.o_buf;
                a.pprev = rec_w ? pprev : nullptr;
                a.aprev = last ? b.aprev : nullptr;
                if (Kp > 0 || n_proxies(&p) > 0) {
                    // centroid proxies: [batch][K] recorded rows per layer (a step without refresh records none)
                    const size_t Kall = (size_t)n_proxies(&p);
                    a.pprev = rec_w ? b.pprev + (size_t)l * bs * Kall * m.n_heads * N : nullptr;
                    a.cluster_K = (int)Kall;
                }
                a.pprev_lse = b.pprev_lse + (size_t)l * bs * (n_proxies(&p) ? (size_t)n_proxies(&p) : (size_t)Wm) * m.n_heads;
                a.aprev_lse = b.aprev_lse;
                a.kl = b.kl; a.N = N; a.n_heads = m.n_heads; a.n_kv = m.n_kv_heads; a.head_dim = m.head_dim;
                a.W_max = Wm; a.B = B; a.record_kl = sd.record_kl; a.rows_per_seq = sd.rows_per_seq; a.batch = bs;
                a.scale = 1.0f / sqrtf((float)m.head_dim);
                // positions whose K/V this layer's QKV projection writes: the forwarded rows of an entry step; the
                // active block and, on refresh steps, the patched window rows of a within-block step
                if (!within) { a.dirty_lo = sd.e0; a.dirty_hi = sd.e0 + sd.rows_per_seq; }
                else {
                    a.dirty_lo = sparse ? std::min(sd.act_start, sd.pre_start) : sd.act_start;
                    a.dirty_hi = sparse ? std::max(sd.act_start + B, sd.suf_start + (sd.W - sd.n_pre)) : sd.act_start + B;
                }
                if ((rc = attention(c, a))) return rc;
            }
            const int* list = nullptr;
            const int* m2_count = nullptr;
            // One sequence with a small window on the tensor-core path: the selection rides on the O projection
            // (idle warps of its first CTA), off the critical path; otherwise it is a kernel of its own.
            const bool sel_in_gemm = sparse && bs == 1 && sd.W <= SEL_SMALL_W && is_bf16 && !(p.flags & POLESTAR_FLAG_SIMT_GEMM) &&
                                     dq % 64 == 0 && d % 256 == 0 && c->sw.fuse_select && Kp == 0;
            tc::SelFuse sf;
            memset(&sf, 0, sizeof(sf));
            if (sparse) {
                Scope sc(c, POLESTAR_PROF_SELECT, (double)bs * sd.W * (m.n_heads * 4 + 8), 0, sel_in_gemm ? 0 : 1);
                StepSelArgs s;
                memset(&s, 0, sizeof(s));
                s.kl = b.kl; s.drift = b.drift + (size_t)l * bs * Wm; s.sel_idx = b.sel_idx + (size_t)l * bs * Wm;
                s.sel_cnt = b.sel_cnt + (size_t)l * bs; s.flag_next = b.patch + (size_t)(l + 1) * bs * Wm;
                s.forced_idx = b.forced_idx + (size_t)l * bs * Wm; s.forced_cnt = b.forced_cnt + (size_t)l * bs;
                s.list = b.list; s.list_count = b.list_count; s.stats = b.stats; s.n_heads = m.n_heads;
                s.mode = p.select_mode;
                s.k = p.select_mode == POLESTAR_SELECT_TOPK_FRAC ? (int)floorf(p.select_frac * (float)sd.W + 0.5f) : p.select_k;
                s.W_max = Wm; s.thresh = p.select_thresh; s.floor_ = p.drift_floor;
                s.ct = ct; s.cluster_k = p.cluster_k;
                if (sel_in_gemm) { sf.on = 1; sf.sd = sd; sf.a = s; }
                else {
                    CK(launch_k(step_select_kernel, dim3(bs), dim3(SEL_THREADS), 0, st, sd, s));
                    CK(cudaGetLastError());
                }
                list = b.list; m2_count = b.list_count;
            }
            // O projection -> RMSNorm -> gate/up -> down as one persistent kernel when the step is small enough
            bool chained = false;
            // (one sequence: its proxy rows are the last rows of the step and need nothing after the attention scores,
            // so a refresh step with proxies still fits the chained kernel's single row tile)
            const int Mc = (bs == 1 && Kp > 0 && list) ? M - Kp : M;
            if (is_bf16 && !(p.flags & POLESTAR_FLAG_SIMT_GEMM) && Mc <= tc::BLOCK_T && c->sw.chain) {
                ChainSpec sp[4];
                memset(sp, 0, sizeof(sp));
                // (in-place variant: the product is added onto the residual rows themselves, x doubles as x1)
                const bool acc = c->sw.accumulate && !fold;
                float* x1 = acc ? b.x : b.x1;
                sp[0].A = b.o_buf; sp[0].W = c->wo[l]; sp[0].N_out = d; sp[0].K = dq; sp[0].epi = EPI_RESID; sp[0].norm_after = 1;
                sp[0].e.resid = b.x; sp[0].e.out_f32 = x1; sp[0].e.ld_out = d; sp[0].e.accumulate = acc ? 1 : 0;
                sp[0].post.kind = 1; sp[0].post.n_rows = Mc; sp[0].post.d = d; sp[0].post.eps = m.rms_eps; sp[0].post.gain = c->n2[l];
                sp[0].post.a_out = b.a_buf; sp[0].post.x = x1; sp[0].post.list = list; sp[0].post.m_count = m2_count;
                if (acc && list) { sp[0].post.rows = b.rows; sp[0].post.packet = b.packet; sp[0].post.sd = sd; }     // packet rows <- residual rows
                sp[1].A = b.a_buf; sp[1].W = c->wgu[l]; sp[1].N_out = 2 * F; sp[1].K = d; sp[1].epi = EPI_SWIGLU;
                sp[1].e.out_t = b.g_buf; sp[1].e.ld_out = F; sp[1].e.m_count = m2_count;
                sp[2].A = b.g_buf; sp[2].W = c->wd[l]; sp[2].N_out = d; sp[2].K = F; sp[2].epi = EPI_DOWN;
                sp[2].e.rows = b.rows; sp[2].e.list = list; sp[2].e.m_count = m2_count; sp[2].e.resid = x1; sp[2].e.out_f32 = b.x;
                sp[2].e.accumulate = acc ? 1 : 0;
                sp[2].e.packet = b.packet; sp[2].e.W_max = Wm; sp[2].e.within = within; sp[2].e.ld_out = d;
                if (fold) {
                    sp[0].norm_after = 0;
                    sp[0].e.fold_a = b.a_buf; sp[0].e.fold_gain = c->n2[l]; sp[0].e.fold_ss = b.fold_ss + (size_t)(2 * l + 1) * Mm;
                    sp[1].e.in_ss = sp[0].e.fold_ss; sp[1].e.in_eps = m.rms_eps; sp[1].e.in_d = d;
                    if (l + 1 < L) {
                        sp[2].e.fold_a = b.a_buf; sp[2].e.fold_gain = c->n1[l + 1]; sp[2].e.fold_ss = b.fold_ss + (size_t)(2 * l + 2) * Mm;
                    }
                }
                const double by = ((double)d * dq + 3.0 * F * d) * esd, fl = 2.0 * Mc * d * (double)dq + 6.0 * Mlive * F * (double)d;
                // ... and, behind it, the next layer's input staging and QKV projection
                int n_chain = 3;
                double by4 = 0, fl4 = 0;
                // (off by default: measured 1 % slower than launching that projection on its own)
                if (l + 1 < L && !fold && c->sw.chain_qkv && n_proxies(&p) == 0) {      // (proxy rows are staged from the next
                                                                                          // layer's cluster tables, made after this point)
                    n_chain = 4;
                    sp[2].norm_after = 2;
                    PostArgs& po = sp[2].post;
                    po.kind = 2; po.n_rows = M; po.d = d; po.eps = m.rms_eps; po.gain = c->n1[l + 1]; po.a_out = b.a_buf;
                    po.x = b.x; po.rows = b.rows; po.hc = b.hc + (size_t)(l + 1) * bs * Wm * d; po.packet = b.packet;
                    po.patch = b.patch + (size_t)(l + 1) * bs * Wm; po.kvflag = b.kvflag; po.sd = sd;
                    sp[3].A = b.a_buf; sp[3].W = c->wqkv[l + 1]; sp[3].N_out = dq + 2 * dkv; sp[3].K = d; sp[3].epi = EPI_QKV;
                    EpiArgs& eq = sp[3].e;
                    eq.rows = b.rows; eq.kvflag = b.kvflag; eq.rope = b.rope; eq.q_out = b.q_buf;
                    eq.kc = b.kc + (size_t)(l + 1) * bs * N * dkv * es; eq.vc = b.vc + (size_t)(l + 1) * bs * N * dkv * es;
                    eq.N_seq = N; eq.n_heads = m.n_heads; eq.n_kv = m.n_kv_heads; eq.head_dim = m.head_dim; eq.W_max = Wm;
                    eq.within = within; eq.ld_out = dq;
                    by4 = (double)(dq + 2 * dkv) * d * esd; fl4 = 2.0 * M * (double)(dq + 2 * dkv) * d;
                }
                {
                    Scope sc(c, POLESTAR_PROF_GEMM_GATE_UP, by + (n_chain == 4 ? by4 : 0), fl + (n_chain == 4 ? fl4 : 0), 0);
                    if ((rc = launch_gemm_chain<__nv_bfloat16>(c->maps, c->gws, sp, n_chain, Mc, st, sf.on ? &sf : nullptr, &chained))) return rc;
                    if (!chained && n_chain == 4) {
                        n_chain = 3;
                        sp[2].norm_after = 0;
                        if ((rc = launch_gemm_chain<__nv_bfloat16>(c->maps, c->gws, sp, 3, Mc, st, sf.on ? &sf : nullptr, &chained))) return rc;
                    }
                }
                if (chained) { c->launches += 1; qkv_done = (n_chain == 4); }
            }
            // (separate launches, tensor-core path: the same in-place accumulation of the split tiles as in the chained kernel)
            const bool acc_sk = c->sw.accumulate && !fold && is_bf16 && !(p.flags & POLESTAR_FLAG_SIMT_GEMM) && d % 256 == 0 && dq % 64 == 0 && F % 64 == 0;
            float* const x1s = acc_sk ? b.x : b.x1;
            if (!chained) {
            {
                Scope sc(c, POLESTAR_PROF_GEMM_O, (double)d * dq * esd + (double)M * dq * esd + 2.0 * M * d * 4, 2.0 * M * d * (double)dq, 1);
                memset(&e, 0, sizeof(e));
                e.resid = b.x; e.out_f32 = x1s; e.ld_out = d; e.accumulate = acc_sk ? 1 : 0;
                if (fold) { e.fold_a = b.a_buf; e.fold_gain = c->n2[l]; e.fold_ss = b.fold_ss + (size_t)(2 * l + 1) * Mm; }
                PostArgs po;
                memset(&po, 0, sizeof(po));
                po.kind = 1; po.n_rows = M; po.d = d; po.eps = m.rms_eps; po.gain = c->n2[l]; po.a_out = b.a_buf;
                po.x = x1s; po.list = list; po.m_count = m2_count;
                if (acc_sk && list) { po.rows = b.rows; po.packet = b.packet; po.sd = sd; }
                if ((rc = gemm<EPI_RESID>(c, b.o_buf, c->wo[l], M, d, dq, e, &po, &ffn_staged, sf.on ? &sf : nullptr))) return rc;
            }
            if (fold) ffn_staged = true;
            if (!ffn_staged) {
                Scope sc(c, POLESTAR_PROF_STAGE, Mlive * d * (4 + esd), 0, 1);
                CK(launch_k(prep_rows_kernel<T>, dim3(M), dim3(norm_threads(M, d)), 0, st, x1s, list, m2_count, c->n2[l], m.rms_eps, d, (T*)b.a_buf,
                            (acc_sk && list) ? b.rows : (const Row*)nullptr, (acc_sk && list) ? b.packet : (float*)nullptr, Wm));
                CK(cudaGetLastError());
            }
            {
                Scope sc(c, POLESTAR_PROF_GEMM_GATE_UP, (2.0 * F * d + Mlive * d + Mlive * F) * esd, 4.0 * Mlive * F * (double)d, 1);
                memset(&e, 0, sizeof(e));
                e.out_t = b.g_buf; e.ld_out = F; e.m_count = m2_count;
                if (fold) { e.in_ss = b.fold_ss + (size_t)(2 * l + 1) * Mm; e.in_eps = m.rms_eps; e.in_d = d; }
                if ((rc = gemm<EPI_SWIGLU>(c, b.a_buf, c->wgu[l], M, 2 * F, d, e))) return rc;
            }
            {
                Scope sc(c, POLESTAR_PROF_GEMM_DOWN, ((double)F * d + Mlive * F) * esd + 2.0 * Mlive * d * 4, 2.0 * Mlive * F * (double)d, 1);
                memset(&e, 0, sizeof(e));
                e.rows = b.rows; e.list = list; e.m_count = m2_count; e.resid = x1s; e.out_f32 = b.x; e.packet = b.packet;
                e.W_max = Wm; e.within = within; e.ld_out = d; e.accumulate = acc_sk ? 1 : 0;
                if (fold && l + 1 < L) { e.fold_a = b.a_buf; e.fold_gain = c->n1[l + 1]; e.fold_ss = b.fold_ss + (size_t)(2 * l + 2) * Mm; }
                PostArgs po;
                memset(&po, 0, sizeof(po));
                if (l + 1 < L && n_proxies(&p) == 0) {
                    po.kind = 2; po.n_rows = M; po.d = d; po.eps = m.rms_eps; po.gain = c->n1[l + 1]; po.a_out = b.a_buf;
                    po.x = b.x; po.rows = b.rows; po.hc = b.hc + (size_t)(l + 1) * bs * Wm * d; po.packet = b.packet;
                    po.patch = b.patch + (size_t)(l + 1) * bs * Wm; po.kvflag = b.kvflag; po.sd = sd;
                }
                if ((rc = gemm<EPI_DOWN>(c, b.g_buf, c->wd[l], M, d, F, e, &po, &qkv_staged))) return rc;
            }
            }
        }
        if (p.flags & POLESTAR_FLAG_KEEP_HIDDEN) {
            Scope sc(c, POLESTAR_PROF_MISC, 0, 0, 1);
            CK(launch_k(keep_hidden_kernel, dim3(bs * B), dim3(256), 0, st, sd, b.x, act_off, d, b.hidden_keep + (size_t)L * bs * B * d));
        }

        // logits of the active rows (+ eligible suffix rows), confidences
        const int use_suffix = sparse && (p.flags & POLESTAR_FLAG_SUFFIX_COMMIT);
        const int Mh = use_suffix ? c->rows_lm : bs * B;
        {
            Scope sc(c, POLESTAR_PROF_STAGE, (double)bs * B * d * (4 + esd), 0, 2);
            CK(launch_k(build_head_list_kernel, dim3(1), dim3(256), 0, st, sd, b.y, m.mask_id, b.sel_idx + (size_t)(L - 1) * bs * Wm,
                                                      b.sel_cnt + (size_t)(L - 1) * bs, use_suffix, 0, b.head_list,
                                                      b.head_count, b.suf_seq, b.suf_w));
            CK(launch_k(prep_head_kernel<T>, dim3(Mh), dim3(norm_threads(Mh, d)), 0, st, b.x, b.packet, b.head_list, b.head_count, c->final_norm, m.rms_eps, d,
                                                   (T*)b.a_head));
            CK(cudaGetLastError());
        }
        {
            Scope sc(c, POLESTAR_PROF_GEMM_LM_HEAD, ((double)m.vocab * d + (double)bs * B * d) * esd + (double)bs * B * m.vocab * 4,
                     2.0 * bs * B * (double)m.vocab * d, 1);
            EpiArgs e;
            memset(&e, 0, sizeof(e));
            e.out_f32 = b.logits; e.ld_out = m.vocab; e.scale = p.logit_scale; e.m_count = b.head_count;
            if ((rc = gemm<EPI_LOGITS>(c, b.a_head, c->lm_head, Mh, m.vocab, d, e))) return rc;
        }
        {
            Scope sc(c, POLESTAR_PROF_CONFIDENCE, (double)bs * B * m.vocab * 4, 0, 3);
            CK(launch_k(conf_partial_kernel, dim3(CONF_CHUNKS, Mh), dim3(256), 0, st, b.logits, b.head_count, Mh, m.vocab, m.mask_id,
                                                                      CONF_CHUNKS, b.conf_part));
            CK(launch_k(conf_final_kernel, dim3((Mh + 127) / 128), dim3(128), 0, st, b.conf_part, b.head_count, Mh, CONF_CHUNKS, b.yhat, b.conf));
            CK(launch_k(delta_kernel, dim3(bs), dim3(256), 0, st, sd, b.kl, act_off, m.n_heads, b.delta));
            CK(cudaGetLastError());
        }
        c->last_act_row_off = act_off;
        return POLESTAR_OK;
    }
};

static StepDesc make_step_desc(polestar_ctx* c, bool* any_refresh) {
    const polestar_params& p = c->p;
    StepDesc sd;
    memset(&sd, 0, sizeof(sd));
    const int N = c->N, B = c->B;
    const bool nocache = (p.flags & POLESTAR_FLAG_NOCACHE) != 0;
    const int start = p.prompt_len + c->block * B, end = start + B;
    sd.batch = p.batch; sd.N = N; sd.B = B; sd.act_start = start; sd.W_max = c->W_max;
    const int Kp = n_proxies(&p);
    sd.pre_start = (int)std::max<long long>(0, (long long)start - (long long)p.win_prefix_blocks * B);
    sd.n_pre = start - sd.pre_start;
    sd.suf_start = end;
    const int n_suf = (int)(std::min<long long>(N, (long long)end + (long long)p.win_suffix_blocks * B) - end);
    sd.W = sd.n_pre + n_suf;
    *any_refresh = false;
    if (c->need_entry || nocache) {
        const bool full = nocache || (c->block % p.full_entry_period == 0);
        sd.kind = full ? 0 : 1;
        sd.e0 = full ? 0 : sd.pre_start;
        sd.rows_per_seq = (full ? N : (sd.n_pre + B + n_suf)) + Kp;
        sd.K = Kp;
        sd.within = 0;
        sd.record_kl = (nocache && !c->need_entry) ? 1 : 0;
    } else {
        sd.kind = 2;
        sd.within = 1;
        sd.record_kl = 1;
        for (int s = 0; s < p.batch; ++s) {
            const bool r = p.tau_upd < 0 || c->cum[s] > p.tau_upd;
            sd.refresh.v[s] = r ? 1 : 0;
            if (r) { *any_refresh = true; c->cum[s] = 0; }
        }
        sd.K = *any_refresh ? Kp : 0;
        sd.rows_per_seq = *any_refresh ? B + sd.W + Kp : B;
    }
    return sd;
}

extern "C" int polestar_step(polestar_ctx* c, polestar_step_info* info) {
    if (!c) return POLESTAR_E_INVAL;
    if (c->failed) return POLESTAR_E_STATE;
    if (c->done) return POLESTAR_E_DONE;
    if (c->pending) return POLESTAR_E_STATE;
    bool any_refresh = false;
    StepDesc sd = make_step_desc(c, &any_refresh);
    int rc = c->m.dtype == POLESTAR_BF16 ? Path<__nv_bfloat16>::forward(c, sd, any_refresh)
                                         : Path<float>::forward(c, sd, any_refresh);
    if (rc) return rc;
    if (c->forced_select) {
        CK(cudaMemsetAsync(c->b.forced_cnt, 0xFF, (size_t)c->m.n_layers * c->p.batch * sizeof(int), c->st));
        c->forced_select = false;
    }
    if (c->forced_codes) {                        // imposed codes serve one forward
        CK(cudaMemsetAsync(c->b.fmask, 0, (size_t)c->m.n_layers * c->p.batch * c->W_max, c->st));
        c->forced_codes = false;
    }
    if (c->forced_labels && sd.kind != 2) {       // forced labels serve one block-entry forward
        CK(cudaMemsetAsync(c->b.forced_labels, 0xFF, (size_t)c->m.n_layers * c->p.batch * c->W_max * sizeof(int), c->st));
        c->forced_labels = false;
    }
    c->last_sd = sd;
    c->pending = true;
    c->forwards += 1;
    if (info) {
        info->kind = sd.kind;
        info->block_index = c->block;
        int nr = 0;
        for (int s = 0; s < c->p.batch; ++s) nr += sd.refresh.v[s];
        info->n_refreshing = nr;
        info->rows = sd.rows_per_seq;
        info->forwards = c->forwards;
    }
    return POLESTAR_OK;
}

extern "C" int polestar_commit(polestar_ctx* c, polestar_commit_info* info) {
    if (!c) return POLESTAR_E_INVAL;
    if (c->failed || !c->pending) return POLESTAR_E_STATE;
    const polestar_params& p = c->p;
    const StepDesc& sd = c->last_sd;
    Buffers& b = c->b;
    CommitArgs a;
    memset(&a, 0, sizeof(a));
    a.y = b.y; a.conf = b.conf; a.yhat = b.yhat;
    a.kl = b.kl; a.delta_out = b.delta; a.Delta_out = b.Delta; a.taud_out = b.taud;
    a.theta = b.theta; a.theta_cnt = b.theta_cnt; a.commit_flags = b.commit_flags; a.own_flags = b.own_flags;
    a.suffix_flags = b.suffix_flags;
    a.head_count = b.head_count; a.suf_seq = b.suf_seq; a.suf_w = b.suf_w;
    a.forced_pos = c->forced_commit ? b.forced_commit : nullptr;
    a.forced_n = c->forced_commit_n;
    a.forced_tok = (c->forced_commit && c->forced_tokens) ? b.forced_tok : nullptr;
    a.seq_info = b.seq_info; a.stats = b.stats; a.status = b.status; a.batch = p.batch;
    a.n_heads = c->m.n_heads; a.hist = p.hist; a.mask_id = c->m.mask_id; a.eos_id = c->m.eos_id;
    a.act_row_off = c->last_act_row_off; a.steps_used = c->steps_used;
    a.steps_per_block = std::max(1, p.max_steps / std::max(1, c->n_blocks));
    a.use_drift = (p.flags & POLESTAR_FLAG_DRIFT_COMMIT) ? 1 : 0;
    a.use_suffix = (p.flags & POLESTAR_FLAG_SUFFIX_COMMIT) ? 1 : 0;
    a.ge = (p.flags & POLESTAR_FLAG_GE_COMPARE) ? 1 : 0;
    a.tau_s = p.tau_s; a.alpha = p.alpha; a.tau_suffix = p.tau_suffix;
    const bool entry_like = sd.record_kl == 0;
    if (entry_like) CK(cudaMemsetAsync(b.theta_cnt, 0, p.batch * sizeof(int), c->st));   // history cleared at block entry
    {
        Scope sc(c, POLESTAR_PROF_COMMIT, (double)p.batch * c->B * 16, 0, 1);
        CK(launch_k(commit_kernel, dim3(p.batch), dim3(256), 0, c->st, sd, a));
        CK(cudaGetLastError());
    }
    if (!c->seq_info_host && cudaHostAlloc((void**)&c->seq_info_host, ((size_t)p.batch * 8 + 8) * sizeof(int), cudaHostAllocDefault) != cudaSuccess)
        return POLESTAR_E_CUDA;
    CK(cudaMemcpyAsync(c->seq_info_host, b.seq_info, ((size_t)p.batch * 8 + 8) * sizeof(int), cudaMemcpyDeviceToHost, c->st));
    CK(cudaStreamSynchronize(c->st));
    for (const auto& r : c->prof_recs) {
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, c->prof_ev[r.ev], c->prof_ev[r.ev + 1]) == cudaSuccess) {
            c->prof_acc[r.fam][0] += 1; c->prof_acc[r.fam][1] += ms;
            c->prof_acc[r.fam][2] += r.bytes; c->prof_acc[r.fam][3] += r.flops;
        }
    }
    c->prof_recs.clear();
    c->prof_used = 0;
    c->pending = false;
    c->forced_commit = false;
    c->forced_tokens = false;
    const int* si = c->seq_info_host;
    polestar_commit_info ci;
    memset(&ci, 0, sizeof(ci));
    bool all_block_done = true;
    int nonfinite = 0;
    for (int s = 0; s < p.batch; ++s) {
        const int* o = si + s * 8;
        ci.n_committed += o[0]; ci.n_by_conf += o[1]; ci.n_by_drift += o[2]; ci.n_by_quota += o[3];
        ci.n_suffix += o[4]; ci.n_eos += o[5];
        if (o[6] > 0) all_block_done = false;
        nonfinite += o[7];
        if (entry_like && !(p.flags & POLESTAR_FLAG_NOCACHE)) c->cum[s] = o[0];
        else c->cum[s] += o[0];
    }
    ci.rows_refreshed = si[p.batch * 8];
    const int status = si[p.batch * 8 + 4];
    ci.block_index = c->block;
    c->steps_used += 1;
    c->need_entry = false;
    c->generated += ci.n_committed;
    c->generated_non_eos += ci.n_committed - ci.n_eos;
    if (all_block_done) {
        c->block += 1;
        c->need_entry = true;
        c->steps_used = 0;
        ci.block_done = 1;
        if (c->block >= c->n_blocks) { c->done = true; ci.all_done = 1; }
    }
    ci.forwards = c->forwards; ci.generated = c->generated; ci.generated_non_eos = c->generated_non_eos;
    ci.launches = c->launches;
    if (info) *info = ci;
    if (status) {
        // a bounded device-side wait gave up: tile and grid counters no longer match the host's bookkeeping and
        // outputs may be partial, so the context refuses further work
        c->failed = true;
        return POLESTAR_E_TIMEOUT;
    }
    if (nonfinite) return POLESTAR_E_NONFINITE;
    return POLESTAR_OK;
}

extern "C" int polestar_init(polestar_ctx** out, const polestar_model* m, const polestar_weights* w,
                             const polestar_params* p, const int32_t* prompt, void* ws, size_t ws_bytes, void* stream) {
    if (out) *out = nullptr;
    if (!out || !m || !w || !p || !ws || (!prompt && p->prompt_len > 0)) return POLESTAR_E_INVAL;
    if (!valid_cfg(m, p)) return POLESTAR_E_INVAL;
    if (!w->embed || !w->lm_head || !w->final_norm || !w->wqkv || !w->wo || !w->w_gate_up || !w->w_down || !w->norm1 ||
        !w->norm2)
        return POLESTAR_E_INVAL;
    if (((uintptr_t)ws) & 255) return POLESTAR_E_INVAL;
    const bool prompt_dev = (p->flags & POLESTAR_FLAG_PROMPT_DEVICE) != 0;
    if (!prompt_dev)
        for (int i = 0; i < p->batch * p->prompt_len; ++i)
            if (prompt[i] < 0 || prompt[i] >= m->vocab || prompt[i] == m->mask_id) return POLESTAR_E_INVAL;
    const size_t need = make_plan(m, p, nullptr, nullptr);
    char* ws_aligned = (char*)(((uintptr_t)ws + 1023) & ~(uintptr_t)1023);
    if ((size_t)(ws_aligned - (char*)ws) + need > ws_bytes) return POLESTAR_E_NOSPACE;
    DevInfo di;
    int rc = device_info(&di);
    if (rc) return rc;
    polestar_ctx* c = new (std::nothrow) polestar_ctx();
    if (!c) return POLESTAR_E_INVAL;
    c->m = *m; c->p = *p;
    c->sw = read_switches();
    {
        std::lock_guard<std::mutex> lk(g_mu);
        g_sw = c->sw; g_sw_loaded = true;
        g_use_pdl = c->sw.pdl != 0;
    }
    c->sms = di.sm_count;
    c->maps.l2promo = c->sw.l2promo;
    cudaGetDevice(&c->device);
    for (int l = 0; l < m->n_layers; ++l) {
        if (!w->wqkv[l] || !w->wo[l] || !w->w_gate_up[l] || !w->w_down[l] || !w->norm1[l] || !w->norm2[l]) {
            delete c;
            return POLESTAR_E_INVAL;
        }
        c->wqkv.push_back(w->wqkv[l]); c->wo.push_back(w->wo[l]); c->wgu.push_back(w->w_gate_up[l]);
        c->wd.push_back(w->w_down[l]); c->n1.push_back(w->norm1[l]); c->n2.push_back(w->norm2[l]);
    }
    c->embed = w->embed; c->lm_head = w->lm_head; c->final_norm = w->final_norm;
    c->st = (cudaStream_t)stream;
    c->ws = ws_aligned;
    make_plan(m, p, &c->b, c->ws);
    c->es = m->dtype == POLESTAR_BF16 ? 2 : 4;
    c->N = p->prompt_len + p->gen_len; c->B = p->block; c->W_max = window_max(p);
    c->n_blocks = p->gen_len / p->block;
    c->M_max = p->batch * (std::max(c->N, c->B + c->W_max) + n_proxies(p));
    c->rows_lm = p->batch * (c->B + std::min(p->win_suffix_blocks * c->B, c->W_max));
    c->cum.assign(p->batch, 0);
    c->gws.partial = c->b.gemm_partial; c->gws.partial_bytes = GEMM_PARTIAL_BYTES;
    // the last 512 words of the counter array hold the grid-wide counters, the rest the per-tile counters
    c->gws.counters = c->b.gemm_counters; c->gws.n_counters = GEMM_COUNTERS - 512; c->gws.status = c->b.status;
    c->gws.post_counter = reinterpret_cast<unsigned*>(c->b.gemm_counters + GEMM_COUNTERS - 1); c->gws.post_total = 0;
    c->gws.chain_counter = reinterpret_cast<unsigned*>(c->b.gemm_counters + GEMM_COUNTERS - 512); c->gws.chain_total = 0;
    c->gws.sms = c->sms; c->gws.sw = c->sw; c->gws.pairs = di.gemm_pairs;

    auto fail = [&](int code) { delete c; return code; };
    // zero the persistent state (everything in front of the scratch rows)
    const size_t persist = (size_t)((char*)c->b.rows - c->ws);
    if (cudaMemsetAsync(c->ws, 0, persist, c->st) != cudaSuccess) return fail(POLESTAR_E_CUDA);
    if (cudaMemsetAsync(c->b.forced_cnt, 0xFF, (size_t)m->n_layers * p->batch * sizeof(int), c->st) != cudaSuccess)
        return fail(POLESTAR_E_CUDA);
    if (cudaMemsetAsync(c->b.gemm_counters, 0, GEMM_COUNTERS * sizeof(int), c->st) != cudaSuccess) return fail(POLESTAR_E_CUDA);
    if (n_proxies(p) && cudaMemsetAsync(c->b.forced_labels, 0xFF, (size_t)m->n_layers * p->batch * c->W_max * sizeof(int), c->st) != cudaSuccess)
        return fail(POLESTAR_E_CUDA);
    if (prompt_dev) {
        init_tokens_kernel<<<(p->batch * c->N + 255) / 256, 256, 0, c->st>>>(c->b.y, prompt, p->batch, p->prompt_len, c->N,
                                                                            m->mask_id, m->vocab);
    } else {
        std::vector<int> y((size_t)p->batch * c->N, m->mask_id);
        for (int s = 0; s < p->batch; ++s)
            for (int i = 0; i < p->prompt_len; ++i) y[(size_t)s * c->N + i] = prompt[(size_t)s * p->prompt_len + i];
        if (cudaMemcpyAsync(c->b.y, y.data(), y.size() * sizeof(int), cudaMemcpyHostToDevice, c->st) != cudaSuccess)
            return fail(POLESTAR_E_CUDA);
    }
    const int half = m->head_dim / 2;
    rope_table_kernel<<<(c->N * half + 255) / 256, 256, 0, c->st>>>(c->b.rope, c->N, half, (double)m->rope_theta);
    if (cudaStreamSynchronize(c->st) != cudaSuccess) return fail(POLESTAR_E_CUDA);
#ifdef POLESTAR_TRACE
    if (c->sw.kernel_trace) {
        long long* tb = (long long*)((char*)c->b.gemm_partial + GEMM_PARTIAL_BYTES - 16384 - 65536);
        cudaMemsetAsync(tb, 0, 65536, c->st);
        cudaMemcpyToSymbolAsync(g_trace_buf, &tb, sizeof(tb), 0, cudaMemcpyHostToDevice, c->st);
        c->trace_installed = true;
    }
#endif
    rc = polestar_step(c, nullptr);
    if (rc) return fail(rc);
    *out = c;
    return POLESTAR_OK;
}

extern "C" void polestar_destroy(polestar_ctx* c) {
    if (!c) return;
    cudaStreamSynchronize(c->st);
#ifdef POLESTAR_TRACE
    if (c->trace_installed) {        // the stamps must not outlive the workspace they are written to
        long long* none = nullptr;
        cudaMemcpyToSymbol(g_trace_buf, &none, sizeof(none));
    }
#endif
    for (cudaEvent_t e : c->prof_ev) cudaEventDestroy(e);
    if (c->seq_info_host) cudaFreeHost(c->seq_info_host);
    delete c;
}

extern "C" int polestar_profile(polestar_ctx* c, double* out, int32_t reset) {
    if (!c || !out) return POLESTAR_E_INVAL;
    memcpy(out, c->prof_acc, sizeof(c->prof_acc));
    if (reset) memset(c->prof_acc, 0, sizeof(c->prof_acc));
    return POLESTAR_OK;
}

extern "C" int polestar_tokens(polestar_ctx* c, int32_t* out) {
    if (!c || !out) return POLESTAR_E_INVAL;
    CK(cudaMemcpyAsync(out, c->b.y, (size_t)c->p.batch * c->N * sizeof(int), cudaMemcpyDeviceToHost, c->st));
    CK(cudaStreamSynchronize(c->st));
    return POLESTAR_OK;
}

extern "C" int polestar_read(polestar_ctx* c, int32_t what, int32_t layer, void* dst, size_t bytes) {
    if (!c || !dst) return POLESTAR_E_INVAL;
    const polestar_model& m = c->m;
    const size_t bs = c->p.batch, B = c->B, Wm = c->W_max, N = c->N, d = m.d_model, L = m.n_layers;
    const size_t dkv = (size_t)m.n_kv_heads * m.head_dim;
    const void* src = nullptr;
    size_t sz = 0;
    const bool need_layer = what == POLESTAR_READ_DRIFT || what == POLESTAR_READ_SEL_COUNT || what == POLESTAR_READ_SEL_IDX ||
                            what == POLESTAR_READ_KCACHE || what == POLESTAR_READ_VCACHE || what == POLESTAR_READ_HCACHE ||
                            what == POLESTAR_READ_PPREV;
    if (need_layer && (layer < 0 || layer >= (int)L)) return POLESTAR_E_INVAL;
    switch (what) {
        case POLESTAR_READ_LOGITS: src = c->b.logits; sz = bs * B * m.vocab * 4; break;
        case POLESTAR_READ_CONF: src = c->b.conf; sz = bs * B * 4; break;
        case POLESTAR_READ_YHAT: src = c->b.yhat; sz = bs * B * 4; break;
        case POLESTAR_READ_DELTA: src = c->b.delta; sz = bs * B * 4; break;
        case POLESTAR_READ_DRIFT: src = c->b.drift + layer * bs * Wm; sz = bs * Wm * 4; break;
        case POLESTAR_READ_SEL_COUNT: src = c->b.sel_cnt + layer * bs; sz = bs * 4; break;
        case POLESTAR_READ_SEL_IDX: src = c->b.sel_idx + layer * bs * Wm; sz = bs * Wm * 4; break;
        case POLESTAR_READ_HIDDEN:
            if (!(c->p.flags & POLESTAR_FLAG_KEEP_HIDDEN) || layer < 0 || layer > (int)L) return POLESTAR_E_INVAL;
            src = c->b.hidden_keep + layer * bs * B * d; sz = bs * B * d * 4; break;
        case POLESTAR_READ_KCACHE: src = c->b.kc + layer * bs * N * dkv * c->es; sz = bs * N * dkv * c->es; break;
        case POLESTAR_READ_VCACHE: src = c->b.vc + layer * bs * N * dkv * c->es; sz = bs * N * dkv * c->es; break;
        case POLESTAR_READ_HCACHE:
            if (c->p.flags & POLESTAR_FLAG_NVFP4_HCACHE) {
                // NVFP4 residual cache: reference row of the row's cluster + decoded residual, put together on the host
                const size_t Kp = (size_t)n_proxies(&c->p), n_rows = bs * Wm;
                std::vector<unsigned char> hq(n_rows * (d / 2)), hs(n_rows * (d / 16));
                std::vector<float> z0(bs * Kp * d);
                std::vector<int> lab(n_rows);
                CK(cudaMemcpyAsync(hq.data(), c->b.hq + layer * hq.size(), hq.size(), cudaMemcpyDeviceToHost, c->st));
                CK(cudaMemcpyAsync(hs.data(), c->b.hs + layer * hs.size(), hs.size(), cudaMemcpyDeviceToHost, c->st));
                CK(cudaMemcpyAsync(z0.data(), c->b.z0 + layer * z0.size(), z0.size() * 4, cudaMemcpyDeviceToHost, c->st));
                CK(cudaMemcpyAsync(lab.data(), c->b.labels + layer * n_rows, n_rows * 4, cudaMemcpyDeviceToHost, c->st));
                CK(cudaStreamSynchronize(c->st));
                static const float grid[8] = {0.f, 0.5f, 1.f, 1.5f, 2.f, 3.f, 4.f, 6.f};
                float* o = (float*)dst;
                const size_t n_out = std::min(n_rows * d, bytes / 4);
                for (size_t i = 0; i < n_out; ++i) {
                    const size_t r = i / d, ch = i % d, sq = r / Wm;
                    if (lab[r] < 0) { o[i] = 0.f; continue; }
                    const unsigned sb = hs[r * (d / 16) + ch / 16], e = (sb >> 3) & 15u, mm = sb & 7u;
                    const float sc = e == 0 ? (float)mm * 0.001953125f : ldexpf(1.f + (float)mm * 0.125f, (int)e - 7);
                    const unsigned code = (hq[r * (d / 2) + ch / 2] >> (4 * (ch & 1))) & 15u;
                    const float v = grid[code & 7u] * sc;
                    o[i] = z0[(sq * Kp + (size_t)lab[r]) * d + ch] + ((code & 8u) ? -v : v);
                }
                return POLESTAR_OK;
            }
            src = c->b.hc + layer * bs * Wm * d; sz = bs * Wm * d * 4; break;
        case POLESTAR_READ_COMMIT: src = c->b.commit_flags; sz = bs * B * 4; break;
        case POLESTAR_READ_PPREV: {
            // stored as (row, lse) with log-probability = row - lse: put together on the host
            const size_t n_rows = bs * (n_proxies(&c->p) ? (size_t)n_proxies(&c->p) : Wm) * m.n_heads;
            std::vector<float> rows(n_rows * N), lse(n_rows);
            CK(cudaMemcpyAsync(rows.data(), c->b.pprev + layer * n_rows * N, rows.size() * 4, cudaMemcpyDeviceToHost, c->st));
            CK(cudaMemcpyAsync(lse.data(), c->b.pprev_lse + layer * n_rows, lse.size() * 4, cudaMemcpyDeviceToHost, c->st));
            CK(cudaStreamSynchronize(c->st));
            const size_t n_out = std::min(rows.size(), bytes / 4);
            float* o = (float*)dst;
            for (size_t i = 0; i < n_out; ++i) o[i] = rows[i] - lse[i / N];
            return POLESTAR_OK;
        }
        case POLESTAR_READ_SUFFIX: src = c->b.suffix_flags; sz = bs * Wm * 4; break;
        case POLESTAR_READ_DRIFT_DELTA: src = c->b.Delta; sz = bs * B * 4; break;
        case POLESTAR_READ_TAU_D: src = c->b.taud; sz = bs * B * 4; break;
        case POLESTAR_READ_THETA: src = c->b.theta; sz = bs * std::max<size_t>(1, c->p.hist) * B * 4; break;
        case POLESTAR_READ_THETA_COUNT: src = c->b.theta_cnt; sz = bs * 4; break;
        case POLESTAR_READ_OWN_COMMIT: src = c->b.own_flags; sz = bs * B * 4; break;
        case POLESTAR_READ_LABELS:
            if (!n_proxies(&c->p) || layer < 0 || layer >= (int)L) return POLESTAR_E_INVAL;
            src = c->b.labels + layer * bs * Wm; sz = bs * Wm * 4; break;
#ifdef POLESTAR_TRACE
        case POLESTAR_READ_TRACE_KERNELS: src = (char*)c->b.gemm_partial + GEMM_PARTIAL_BYTES - 16384 - 65536; sz = 65536; break;
        case POLESTAR_READ_TRACE_GEMM: src = (char*)c->b.gemm_partial + GEMM_PARTIAL_BYTES - 16384; sz = 16384; break;
#endif
        default: return POLESTAR_E_INVAL;
    }
    CK(cudaMemcpyAsync(dst, src, std::min(sz, bytes), cudaMemcpyDeviceToHost, c->st));
    CK(cudaStreamSynchronize(c->st));
    return POLESTAR_OK;
}

extern "C" int polestar_force(polestar_ctx* c, int32_t what, int32_t layer, const int32_t* idx, int32_t n) {
    if (!c) return POLESTAR_E_INVAL;
    const int bs = c->p.batch, Wm = c->W_max, L = c->m.n_layers;
    if (what == POLESTAR_FORCE_CLEAR) {
        CK(cudaMemsetAsync(c->b.forced_cnt, 0xFF, (size_t)L * bs * sizeof(int), c->st));
        c->forced_select = false; c->forced_commit = false;
        return POLESTAR_OK;
    }
    if (n < 0 || (n > 0 && !idx)) return POLESTAR_E_INVAL;
    if (what == POLESTAR_FORCE_SELECT) {
        if (layer < 0 || layer >= L || n > Wm) return POLESTAR_E_INVAL;
        std::vector<int> cnt(bs, 0);
        for (int s = 0; s < bs; ++s) {
            int ns = 0;
            while (ns < n && idx[s * n + ns] >= 0) ++ns;       // trailing -1 entries pad shorter lists
            for (int i = 0; i < ns; ++i) {
                const int w = idx[s * n + i];
                if (w >= Wm || (i > 0 && w <= idx[s * n + i - 1])) return POLESTAR_E_INVAL;
            }
            cnt[s] = ns;
            if (ns) CK(cudaMemcpyAsync(c->b.forced_idx + ((size_t)layer * bs + s) * Wm, idx + (size_t)s * n, ns * sizeof(int),
                                       cudaMemcpyHostToDevice, c->st));
        }
        CK(cudaMemcpyAsync(c->b.forced_cnt + (size_t)layer * bs, cnt.data(), bs * sizeof(int), cudaMemcpyHostToDevice, c->st));
        CK(cudaStreamSynchronize(c->st));
        c->forced_select = true;
        return POLESTAR_OK;
    }
    if (what == POLESTAR_FORCE_LABELS) {
        if (!n_proxies(&c->p) || layer < 0 || layer >= L || n <= 0 || n > Wm) return POLESTAR_E_INVAL;
        for (int s = 0; s < bs; ++s)
            CK(cudaMemcpyAsync(c->b.forced_labels + ((size_t)layer * bs + s) * Wm, idx + (size_t)s * n, n * sizeof(int),
                               cudaMemcpyHostToDevice, c->st));
        CK(cudaStreamSynchronize(c->st));
        c->forced_labels = true;
        return POLESTAR_OK;
    }
    if (what == POLESTAR_FORCE_HCODES) {
        const unsigned want = POLESTAR_FLAG_NVFP4_HCACHE | POLESTAR_FLAG_KEEP_HIDDEN;
        if ((c->p.flags & want) != want) return POLESTAR_E_STATE;
        if (layer < 0 || layer >= L || n <= 0 || n > Wm || !idx) return POLESTAR_E_INVAL;
        const size_t d = (size_t)c->m.d_model, W = (size_t)Wm;
        const unsigned char* blob = (const unsigned char*)idx;
        const unsigned char* hm = blob; const unsigned char* hq = hm + (size_t)bs * n; const unsigned char* hs = hq + (size_t)bs * n * (d / 2);
        if (!c->forced_codes) CK(cudaMemsetAsync(c->b.fmask, 0, (size_t)L * bs * W, c->st));
        for (int s = 0; s < bs; ++s) {
            const size_t o = ((size_t)layer * bs + s) * W;
            CK(cudaMemcpyAsync(c->b.fmask + o, hm + (size_t)s * n, n, cudaMemcpyHostToDevice, c->st));
            CK(cudaMemcpyAsync(c->b.fq + o * (d / 2), hq + (size_t)s * n * (d / 2), (size_t)n * (d / 2), cudaMemcpyHostToDevice, c->st));
            CK(cudaMemcpyAsync(c->b.fs + o * (d / 16), hs + (size_t)s * n * (d / 16), (size_t)n * (d / 16), cudaMemcpyHostToDevice, c->st));
        }
        const size_t o = (size_t)layer * bs * W;
        impose_codes_kernel<<<(unsigned)(bs * W), 128, 0, c->st>>>(c->b.fmask + o, c->b.fq + o * (d / 2), c->b.fs + o * (d / 16),
                                                                  c->b.hq + o * (d / 2), c->b.hs + o * (d / 16), (int)d);
        CK(cudaGetLastError());
        CK(cudaStreamSynchronize(c->st));
        c->forced_codes = true;
        return POLESTAR_OK;
    }
    if (what == POLESTAR_FORCE_COMMIT) {
        if (n > FORCED_COMMIT_MAX) return POLESTAR_E_INVAL;
        if (n) CK(cudaMemcpyAsync(c->b.forced_commit, idx, (size_t)bs * n * sizeof(int), cudaMemcpyHostToDevice, c->st));
        CK(cudaStreamSynchronize(c->st));
        c->forced_commit = true;
        c->forced_tokens = false;
        c->forced_commit_n = n;
        return POLESTAR_OK;
    }
    if (what == POLESTAR_FORCE_TOKENS) {
        if (!c->forced_commit || n != c->forced_commit_n) return POLESTAR_E_STATE;
        if (n) CK(cudaMemcpyAsync(c->b.forced_tok, idx, (size_t)bs * n * sizeof(int), cudaMemcpyHostToDevice, c->st));
        CK(cudaStreamSynchronize(c->st));
        c->forced_tokens = true;
        return POLESTAR_OK;
    }
    return POLESTAR_E_INVAL;
}

// ------------------------------------------------------------------------------------------
// single kernels
// ------------------------------------------------------------------------------------------
extern "C" int polestar_k_attention(const void* q, const void* k, const void* v, float* logp_prev, float* lse_prev,
                                    float* kl, void* out, int32_t R, int32_t N, int32_t n_heads, int32_t n_kv,
                                    int32_t head_dim, int32_t dtype, void* stream) {
    if (R < 0 || N <= 0 || n_heads <= 0 || n_kv <= 0 || n_heads % n_kv || head_dim <= 0 || head_dim > 256)
        return POLESTAR_E_INVAL;
    if (dtype != POLESTAR_F32 && dtype != POLESTAR_BF16) return POLESTAR_E_INVAL;
    if (R == 0) return POLESTAR_OK;              // no rows: nothing to do (the row pointers may be null)
    if (!q || !k || !v) return POLESTAR_E_INVAL;
    if (logp_prev && (!kl || !lse_prev)) return POLESTAR_E_INVAL;
    cudaStream_t st = (cudaStream_t)stream;
    AttnArgs a;
    memset(&a, 0, sizeof(a));
    a.n_rows = R; a.q = q; a.kc = k; a.vc = v; a.out = out; a.pprev = logp_prev; a.pprev_lse = lse_prev; a.kl = kl; a.N = N;
    a.n_heads = n_heads; a.n_kv = n_kv; a.head_dim = head_dim; a.record_kl = 1; a.rows_per_seq = R; a.batch = 1;
    a.scale = 1.0f / sqrtf((float)head_dim);
    a.dirty_lo = 0; a.dirty_hi = N;              // a stand-alone call knows nothing about who wrote K / V: wait for everything
    DevInfo di;
    int rc = device_info(&di);
    if (rc) return rc;
    const Switches sw = stand_alone_switches();
    if (dtype == POLESTAR_BF16 && head_dim == 128 && !sw.attn_simt) {
        if (attention_stream_applies(a) && (sw.attn_kernel == 9 || (sw.attn_kernel == 0 && attention_prefers_stream(a))) &&
            !((((uintptr_t)q | (uintptr_t)k | (uintptr_t)v)) & 15)) {
            MapCache maps;
            maps.l2promo = sw.l2promo;
            return launch_attention_stream(maps, a, st, nullptr);
        }
        if ((sw.attn_kernel == 0 || sw.attn_kernel == 8) && attention_tc_applies(a) &&
            !((((uintptr_t)q | (uintptr_t)k | (uintptr_t)v)) & 15)) {
            MapCache maps;                 // the three tensor maps of this call
            maps.l2promo = sw.l2promo;
            return launch_attention_tc(maps, a, st, nullptr);
        }
        CK(launch_attention_mma(a, st, di.sm_count, sw.attn_kernel));
        return POLESTAR_OK;
    }
    const int wpb = 4;
    const size_t smem = (size_t)wpb * N * sizeof(float);
    if (smem > SIMT_ATTN_SMEM_MAX) return POLESTAR_E_INVAL;
    dim3 grid((R + wpb - 1) / wpb, n_heads);
    if (dtype == POLESTAR_BF16) attention_simt_kernel<__nv_bfloat16><<<grid, wpb * 32, smem, st>>>(a);
    else attention_simt_kernel<float><<<grid, wpb * 32, smem, st>>>(a);
    CK(cudaGetLastError());
    return POLESTAR_OK;
}

extern "C" int polestar_k_hidden_delta(const void* a, const void* b, float* out, int32_t rows, int32_t d, int32_t dtype,
                                       void* stream) {
    if (rows < 0 || d <= 0) return POLESTAR_E_INVAL;
    if (dtype != POLESTAR_F32 && dtype != POLESTAR_BF16) return POLESTAR_E_INVAL;
    if (rows == 0) return POLESTAR_OK;           // no rows: nothing to do (the pointers may be null)
    if (!a || !b || !out) return POLESTAR_E_INVAL;
    const int per = dtype == POLESTAR_BF16 ? 8 : 4;
    if (d % per || (((uintptr_t)a | (uintptr_t)b) & 15)) return POLESTAR_E_INVAL;
    DevInfo di;
    int rc = device_info(&di);
    if (rc) return rc;
    const int wpb = 8;
    const int grid = std::min((rows + wpb - 1) / wpb, di.sm_count * 8);
    if (dtype == POLESTAR_BF16)
        hidden_delta_kernel<__nv_bfloat16><<<grid, wpb * 32, 0, (cudaStream_t)stream>>>((const __nv_bfloat16*)a, (const __nv_bfloat16*)b, out, rows, d);
    else
        hidden_delta_kernel<float><<<grid, wpb * 32, 0, (cudaStream_t)stream>>>((const float*)a, (const float*)b, out, rows, d);
    CK(cudaGetLastError());
    return POLESTAR_OK;
}

extern "C" int polestar_k_select(const float* drift, int32_t batch, int32_t W, int32_t mode, int32_t k, float thresh,
                                 float floor_, int32_t* idx, int32_t* count, void* stream) {
    if (batch < 0 || W < 0 || W > SEL_MAX_W || mode < 0 || mode > 4) return POLESTAR_E_INVAL;
    if (batch == 0) return POLESTAR_OK;
    if (!count) return POLESTAR_E_INVAL;
    if (W == 0) {                                 // no candidates: every count is zero (drift and idx may be null)
        CK(cudaMemsetAsync(count, 0, (size_t)batch * sizeof(int32_t), (cudaStream_t)stream));
        return POLESTAR_OK;
    }
    if (!drift || !idx) return POLESTAR_E_INVAL;
    select_kernel<<<batch, SEL_THREADS, 0, (cudaStream_t)stream>>>(drift, W, mode, k, thresh, floor_, idx, count);
    CK(cudaGetLastError());
    return POLESTAR_OK;
}

static size_t refresh_layout(int batch, int max_rows, int d, int head_dim, int P, size_t* off_rope, size_t* off_part,
                             size_t* off_cnt, size_t* off_status) {
    Plan pl;
    pl.take((size_t)batch * max_rows * d * 2 + 256 * (size_t)d * 2);   // staged rows (+ one tile of slack)
    *off_rope = pl.take((size_t)P * (head_dim / 2) * sizeof(float2));
    *off_part = pl.take(GEMM_PARTIAL_BYTES);
    *off_cnt = pl.take(GEMM_COUNTERS * sizeof(int));
    *off_status = pl.take(sizeof(int));
    return pl.total;
}

extern "C" size_t polestar_k_refresh_scratch_bytes(int32_t batch, int32_t max_rows, int32_t d, int32_t n_heads,
                                                   int32_t n_kv, int32_t head_dim) {
    (void)n_heads; (void)n_kv;
    if (batch <= 0 || max_rows <= 0 || d <= 0 || head_dim <= 0) return 0;
    size_t a, b, c, e;
    return refresh_layout(batch, max_rows, d, head_dim, 65536, &a, &b, &c, &e);
}

extern "C" int polestar_k_refresh(const void* h, const int32_t* idx, const int32_t* counts, const void* wqkv,
                                  const float* norm, void* kc, void* vc, void* q_out, int32_t batch, int32_t P,
                                  int32_t max_rows, int32_t d, int32_t n_heads, int32_t n_kv, int32_t head_dim,
                                  float rms_eps, float rope_theta, int32_t dtype, void* scratch, size_t scratch_bytes,
                                  void* stream) {
    if (!h || !idx || !counts || !wqkv || !norm || !kc || !vc || !scratch) return POLESTAR_E_INVAL;
    if (batch <= 0 || P <= 0 || P > 65536 || max_rows <= 0 || max_rows > P || d <= 0 || n_heads <= 0 || n_kv <= 0 ||
        n_heads % n_kv || head_dim <= 0 || head_dim % 2)
        return POLESTAR_E_INVAL;
    if (dtype != POLESTAR_BF16) return POLESTAR_E_INVAL;
    if (((uintptr_t)scratch) & 1023) return POLESTAR_E_INVAL;
    size_t off_rope, off_part, off_cnt, off_status;
    const size_t need = refresh_layout(batch, max_rows, d, head_dim, 65536, &off_rope, &off_part, &off_cnt, &off_status);
    if (scratch_bytes < need) return POLESTAR_E_NOSPACE;
    DevInfo di;
    int rc = device_info(&di);
    if (rc) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    char* sc = (char*)scratch;
    __nv_bfloat16* a_buf = (__nv_bfloat16*)sc;
    float2* rope = (float2*)(sc + off_rope);
    MapCache maps;                     // the two tensor maps of this call (built per call: no shared state)
    GemmWs ws;
    ws.sms = di.sm_count; ws.sw = stand_alone_switches(); ws.pairs = di.gemm_pairs;
    maps.l2promo = ws.sw.l2promo;
    ws.partial = (float*)(sc + off_part); ws.partial_bytes = GEMM_PARTIAL_BYTES;
    const int M = batch * max_rows;
    const int dq = n_heads * head_dim, dkv = n_kv * head_dim;
    // The scratch is caller memory with unknown contents: the split-K tile counters must start at zero.  Only the
    // counters of this GEMM's output tiles (arrivals, then finished shares) are used, so only those are cleared.
    const long long tiles = (long long)((dq + 2 * dkv + tc::BLOCK_F - 1) / tc::BLOCK_F) * ((M + tc::BLOCK_T - 1) / tc::BLOCK_T);
    // (CTA pairs count per 128-row half of their 256-row tiles: up to one more half per feature tile)
    const int n_cnt = (int)std::min<long long>(GEMM_COUNTERS, 2 * (tiles + (dq + 2 * dkv) / tc::BLOCK_F + 2));
    ws.counters = (int*)(sc + off_cnt); ws.n_counters = n_cnt; ws.status = (int*)(sc + off_status);
    const int half = head_dim / 2;
    // Two launches with programmatic stream serialization (the projection starts while the gather drains).  The gather
    // kernel also clears the counters and the status word (read back by polestar_k_refresh_status) and writes the rotary
    // entries of the selected positions; only a refresh of (nearly) every position fills the whole table instead.
    const bool table = M >= P;
    if (table) CK(launch_k(rope_table_kernel, dim3((P * half + 255) / 256), dim3(256), 0, st, rope, P, half, (double)rope_theta));
    CK(launch_k(prep_refresh_kernel<__nv_bfloat16>, dim3(M), dim3(256), 0, st, (const __nv_bfloat16*)h, idx, counts, max_rows, P, norm,
                rms_eps, d, a_buf, table ? (float2*)nullptr : rope, half, (double)rope_theta, ws.counters, n_cnt, ws.status));
    CK(cudaGetLastError());
    EpiArgs e;
    memset(&e, 0, sizeof(e));
    e.rope = rope; e.q_out = q_out; e.kc = kc; e.vc = vc; e.n_heads = n_heads; e.n_kv = n_kv; e.head_dim = head_dim;
    e.idx = idx; e.counts = counts; e.max_rows = max_rows; e.P = P;
    if (d % 64 == 0 && (dq + 2 * dkv) % 256 == 0 && !ws.sw.refresh_simt)
        return launch_gemm_tc<EPI_QKV_REFRESH>(maps, ws, a_buf, wqkv, M, dq + 2 * dkv, d, e, st);
    return launch_gemm_simt<__nv_bfloat16, EPI_QKV_REFRESH>(a_buf, wqkv, M, dq + 2 * dkv, d, e, st);
}

extern "C" int polestar_k_refresh_status(const void* scratch, size_t scratch_bytes, int32_t batch, int32_t max_rows,
                                         int32_t d, int32_t head_dim, void* stream) {
    if (!scratch || batch <= 0 || max_rows <= 0 || d <= 0 || head_dim <= 0) return POLESTAR_E_INVAL;
    size_t off_rope, off_part, off_cnt, off_status;
    const size_t need = refresh_layout(batch, max_rows, d, head_dim, 65536, &off_rope, &off_part, &off_cnt, &off_status);
    if (scratch_bytes < need) return POLESTAR_E_NOSPACE;
    int status = 0;
    CK(cudaMemcpyAsync(&status, (const char*)scratch + off_status, sizeof(int), cudaMemcpyDeviceToHost, (cudaStream_t)stream));
    CK(cudaStreamSynchronize((cudaStream_t)stream));
    return status ? POLESTAR_E_TIMEOUT : POLESTAR_OK;
}

extern "C" int polestar_k_wait_probe(const uint32_t* counter, uint32_t expect, int64_t limit_cycles, int32_t* status, void* stream) {
    if (!counter || !status || limit_cycles <= 0 || limit_cycles > 2000000000LL) return POLESTAR_E_INVAL;
    tc::wait_probe_kernel<<<1, 1, 0, (cudaStream_t)stream>>>(counter, expect, (long long)limit_cycles, status);
    CK(cudaGetLastError());
    int h = 0;
    CK(cudaMemcpyAsync(&h, status, sizeof(int), cudaMemcpyDeviceToHost, (cudaStream_t)stream));
    CK(cudaStreamSynchronize((cudaStream_t)stream));
    return h ? POLESTAR_E_TIMEOUT : POLESTAR_OK;
}

extern "C" int polestar_k_nvfp4_residual(const float* x, const float* ref, int32_t rows, int32_t d, uint8_t* codes,
                                         uint8_t* scales, float* deq, void* stream) {
    if (rows < 0 || d <= 0 || d % 128) return POLESTAR_E_INVAL;
    if (rows == 0) return POLESTAR_OK;
    if (!x || !ref || !codes || !scales || !deq) return POLESTAR_E_INVAL;
    if ((((uintptr_t)x | (uintptr_t)ref | (uintptr_t)deq) & 15) || ((uintptr_t)codes & 1)) return POLESTAR_E_INVAL;
    nvfp4_residual_kernel<<<rows, 256, 0, (cudaStream_t)stream>>>(x, ref, d, codes, scales, deq);
    CK(cudaGetLastError());
    return POLESTAR_OK;
}

// The confidence kernel reads rows with 16-byte loads when the vocabulary is a multiple of four: the base must
// then be 16-byte aligned (rows follow at multiples of 16 bytes); otherwise 4-byte alignment is enough.
static bool conf_logits_aligned(const float* logits, int vocab) {
    return (((uintptr_t)logits) & ((vocab & 3) == 0 ? 15 : 3)) == 0;
}

extern "C" int polestar_k_confidence(const float* logits, int32_t rows, int32_t vocab, int32_t mask_id, int32_t* yhat,
                                     float* conf, void* scratch, size_t scratch_bytes, void* stream) {
    if (rows < 0 || vocab <= 0) return POLESTAR_E_INVAL;
    if (rows == 0) return POLESTAR_OK;           // no rows: nothing to do (the pointers may be null)
    if (!logits || !yhat || !conf || !scratch) return POLESTAR_E_INVAL;
    if (!conf_logits_aligned(logits, vocab)) return POLESTAR_E_INVAL;
    if (scratch_bytes < (size_t)rows * CONF_CHUNKS * sizeof(ConfPart)) return POLESTAR_E_NOSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    conf_partial_kernel<<<dim3(CONF_CHUNKS, rows), 256, 0, st>>>(logits, nullptr, rows, vocab, mask_id, CONF_CHUNKS, (ConfPart*)scratch);
    conf_final_kernel<<<(rows + 127) / 128, 128, 0, st>>>((const ConfPart*)scratch, nullptr, rows, CONF_CHUNKS, yhat, conf);
    CK(cudaGetLastError());
    return POLESTAR_OK;
}

// ------------------------------------------------------------------------------------------
// Confidence without any caller-provided or allocated scratch
// ------------------------------------------------------------------------------------------
// Some callers have no way to obtain device scratch at call time: a serving process that handed
// its whole memory budget to a KV-cache pool at start-up, a latency-critical loop in which
// cudaMalloc's implicit device synchronisation is not acceptable, or a plug-in that is only
// given input and output buffers.  For them the per-chunk partial results of the confidence
// kernel live in a fixed array inside the library image (every GPU that loads the library
// carries these 512 KB until the process exits).
static __device__ __align__(256) ConfPart g_conf_scratch[POLESTAR_NOALLOC_MAX_ROWS * CONF_CHUNKS];

// On the host, `g_conf_scratch` is only a handle of the symbol, not a device address: the real
// address differs per device and has to be looked up once per device with that device current.
static ConfPart* conf_scratch_ptr(int* err) {
    static ConfPart* ptrs[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess || dev < 0 || dev >= 64) { last_cuda_error = e; *err = POLESTAR_E_CUDA; return nullptr; }
    if (!ptrs[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_conf_scratch);
        if (e != cudaSuccess || !p) { last_cuda_error = e; *err = POLESTAR_E_CUDA; return nullptr; }
        ptrs[dev] = (ConfPart*)p;
    }
    *err = POLESTAR_OK;
    return ptrs[dev];
}

extern "C" int polestar_k_confidence_noalloc(const float* logits, int32_t rows, int32_t vocab, int32_t mask_id,
                                             int32_t* yhat, float* conf, void* stream) {
    if (rows < 0 || vocab <= 0) return POLESTAR_E_INVAL;
    if (rows == 0) return POLESTAR_OK;           // no rows: nothing to do (the pointers may be null)
    if (!logits || !yhat || !conf) return POLESTAR_E_INVAL;
    if (!conf_logits_aligned(logits, vocab)) return POLESTAR_E_INVAL;
    if (rows > POLESTAR_NOALLOC_MAX_ROWS) return POLESTAR_E_NOSPACE;    // beyond the built-in scratch: use polestar_k_confidence
    int err = POLESTAR_OK;
    ConfPart* scratch = conf_scratch_ptr(&err);
    if (!scratch) return err;
    cudaStream_t st = (cudaStream_t)stream;
    // every partial the second kernel reads is written by the first one in this call, so nothing of the
    // previous call's contents has to be cleared
    conf_partial_kernel<<<dim3(CONF_CHUNKS, rows), 256, 0, st>>>(logits, nullptr, rows, vocab, mask_id, CONF_CHUNKS, scratch);
    conf_final_kernel<<<(rows + 127) / 128, 128, 0, st>>>(scratch, nullptr, rows, CONF_CHUNKS, yhat, conf);
    CK(cudaGetLastError());
    return POLESTAR_OK;
}
