// Internal declarations shared by the translation units of the SpecBound sm_100a library.
#pragma once
#include <cstdio>
#include <cstdlib>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/specbound.h"

namespace sb {

constexpr int kMaxW = SB_MAX_W;
constexpr int kHeadMaxCtas = 1024;   // upper bound of CTAs of one exit-confidence launch

// ---------------------------------------------------------------------------------------------
// Activation operand of the skinny GEMMs.
//   fp32 models : float [8][K]                      (row i of the round in row i)
//   bf16 models : bf16  [16][K], row i = high part, row 8+i = low part of the fp32 value
//                 (x = hi + lo keeps 16 mantissa bits, so the bf16 tensor-core product of a
//                  weight with an activation is as accurate as an fp32 one)
// ---------------------------------------------------------------------------------------------
template <typename T> struct Act;
template <> struct Act<float> {
    using type = float;
    static constexpr int rows = 8;
    __device__ static void store(float* a, int row, int k, int K, float v) { a[(size_t)row * K + k] = v; }
    __device__ static float load(const float* a, int row, int k, int K) { return a[(size_t)row * K + k]; }
    __device__ static void store4(float* a, int row, int k, int K, float4 v) {
        *reinterpret_cast<float4*>(a + (size_t)row * K + k) = v;
    }
};

// four consecutive gains as floats (k a multiple of 4)
__device__ __forceinline__ float4 load_gain4(const float* g, int k) { return *reinterpret_cast<const float4*>(g + k); }
__device__ __forceinline__ float4 load_gain4(const __nv_bfloat16* g, int k) {
    uint2 u = *reinterpret_cast<const uint2*>(g + k);
    return make_float4(__uint_as_float(u.x << 16), __uint_as_float(u.x & 0xffff0000u), __uint_as_float(u.y << 16),
                       __uint_as_float(u.y & 0xffff0000u));
}
template <> struct Act<__nv_bfloat16> {
    using type = __nv_bfloat16;
    static constexpr int rows = 16;
    __device__ static void store(__nv_bfloat16* a, int row, int k, int K, float v) {
        __nv_bfloat16 hi = __float2bfloat16_rn(v);
        a[(size_t)row * K + k] = hi;
        a[(size_t)(row + 8) * K + k] = __float2bfloat16_rn(v - __bfloat162float(hi));
    }
    __device__ static float load(const __nv_bfloat16* a, int row, int k, int K) {
        return __bfloat162float(a[(size_t)row * K + k]) + __bfloat162float(a[(size_t)(row + 8) * K + k]);
    }
    // four consecutive values (k a multiple of 4): one 8-byte store for the high halves, one for the low halves
    __device__ static void store4(__nv_bfloat16* a, int row, int k, int K, float4 v) {
        __nv_bfloat16 h0 = __float2bfloat16_rn(v.x), h1 = __float2bfloat16_rn(v.y), h2 = __float2bfloat16_rn(v.z),
                      h3 = __float2bfloat16_rn(v.w);
        __nv_bfloat162 hi01 = __halves2bfloat162(h0, h1), hi23 = __halves2bfloat162(h2, h3);
        __nv_bfloat162 lo01 = __halves2bfloat162(__float2bfloat16_rn(v.x - __bfloat162float(h0)),
                                                 __float2bfloat16_rn(v.y - __bfloat162float(h1)));
        __nv_bfloat162 lo23 = __halves2bfloat162(__float2bfloat16_rn(v.z - __bfloat162float(h2)),
                                                 __float2bfloat16_rn(v.w - __bfloat162float(h3)));
        uint2 hp, lp;
        hp.x = *reinterpret_cast<unsigned int*>(&hi01); hp.y = *reinterpret_cast<unsigned int*>(&hi23);
        lp.x = *reinterpret_cast<unsigned int*>(&lo01); lp.y = *reinterpret_cast<unsigned int*>(&lo23);
        *reinterpret_cast<uint2*>(a + (size_t)row * K + k) = hp;
        *reinterpret_cast<uint2*>(a + (size_t)(row + 8) * K + k) = lp;
    }
};

// Programmatic dependent launch.  Every kernel of the library is launched with programmatic
// stream serialisation: it may start while its predecessor is still running, lets its own
// successor start early (pdl_trigger), and must execute pdl_wait -- EVERY thread, before any
// early return -- before it touches memory the predecessor writes or reads.  Only loads of
// weights (never written) may precede the wait.  Without the launch attribute both are no-ops.
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// ---- shared-memory barriers (mbarrier) used by the TMA pipelines ----
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// adds to the bytes the current phase waits for, without arriving
__device__ __forceinline__ void mbar_expect_tx_only(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// plain (untiled) TMA copy of `bytes` (a multiple of 16; both addresses 16-byte aligned) from global to this
// CTA's shared memory, completing on an mbarrier
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst), "l"(src),
                 "r"(bytes), "r"(bar)
                 : "memory");
}

extern bool g_use_pdl;
// With SB_DEBUG set in the environment, CUDA errors are also written to stderr where they are first seen.
inline cudaError_t report_cuda(const char* where, cudaError_t err) {
    if (err != cudaSuccess) {
        static const bool on = getenv("SB_DEBUG") != nullptr;
        if (on) fprintf(stderr, "[specbound] %s: %s (%s)\n", where, cudaGetErrorName(err), cudaGetErrorString(err));
    }
    return err;
}
// Index of the current device for the per-device host-side caches (function attributes, SM count, ...); -1 on error.
constexpr int kMaxDevices = 64;
inline int current_device() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return -1;
    return dev;
}
inline int device_sm_count() {   // SMs of the current device (148 if the query fails)
    static int n[kMaxDevices];
    const int dev = current_device();
    if (dev < 0) return 148;
    if (!n[dev] && (cudaDeviceGetAttribute(&n[dev], cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n[dev] <= 0)) n[dev] = 148;
    return n[dev];
}
// cluster with more than one CTA: launches thread-block clusters of that shape (the grid must be a multiple of it);
// pdl: launch with programmatic stream serialisation (the kernel may start while its predecessor drains)
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kcp(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, dim3 cluster,
                              bool pdl, Args&&... args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[2];
    int n_attr = 0;
    if (pdl) {
        attr[n_attr].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[n_attr].val.programmaticStreamSerializationAllowed = 1;
        ++n_attr;
    }
    if (cluster.x * cluster.y * cluster.z > 1) {
        attr[n_attr].id = cudaLaunchAttributeClusterDimension;
        attr[n_attr].val.clusterDim.x = cluster.x;
        attr[n_attr].val.clusterDim.y = cluster.y;
        attr[n_attr].val.clusterDim.z = cluster.z;
        ++n_attr;
    }
    cfg.attrs = attr;
    cfg.numAttrs = n_attr;
    // every kernel asks for the same (maximal) shared-memory carve-out: an SM never has to drain to
    // change its L1/shared split between two kernels of the chain.  Function attributes are per device.
    static void* seen[kMaxDevices][32];
    static int n_seen[kMaxDevices];
    const int dev = current_device();
    if (dev >= 0) {
        bool known = false;
        for (int i = 0; i < n_seen[dev]; ++i) known |= seen[dev][i] == (void*)kernel;
        if (!known) {
            cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, (int)cudaSharedmemCarveoutMaxShared);
            if (n_seen[dev] < 32) seen[dev][n_seen[dev]++] = (void*)kernel;
        }
    }
    return report_cuda("kernel launch", cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...));
}
// clusters of cluster_y CTAs along y
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kcp(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, int cluster_y,
                              bool pdl, Args&&... args) {
    return launch_kcp(kernel, grid, block, smem, st, dim3(1, cluster_y > 1 ? (unsigned)cluster_y : 1u, 1), pdl, static_cast<Args&&>(args)...);
}
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kc(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, int cluster_y,
                             Args&&... args) {
    return launch_kcp(kernel, grid, block, smem, st, cluster_y, g_use_pdl, static_cast<Args&&>(args)...);
}
template <typename... KArgs, typename... Args>
inline void launch_k(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
    (void)launch_kc(kernel, grid, block, smem, st, 1, static_cast<Args&&>(args)...);
}

__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

constexpr int kMaxSplitK = 8;   // most split-K partials a GEMM leaves for its consumer (= kMaxSplit of the tcgen05 kernels)

// Sum of the split-K partials of one output element, in split order.  All loads are issued before
// the first add (fixed trip count, unused splits predicated off and contributing an exact 0), so a
// consumer pays one L2 round trip instead of one per split.
__device__ __forceinline__ float sum_splits(const float* __restrict__ first, size_t split_stride, int n_split) {
    float v[kMaxSplitK];
#pragma unroll
    for (int s = 0; s < kMaxSplitK; ++s) v[s] = s < n_split ? __ldcg(first + (size_t)s * split_stride) : 0.f;
    float acc = v[0];
#pragma unroll
    for (int s = 1; s < kMaxSplitK; ++s) acc += v[s];
    return acc;
}
__device__ __forceinline__ float2 sum_splits2(const float* __restrict__ first, size_t split_stride, int n_split) {   // two neighbouring elements
    float2 v[kMaxSplitK];
#pragma unroll
    for (int s = 0; s < kMaxSplitK; ++s)
        v[s] = s < n_split ? __ldcg(reinterpret_cast<const float2*>(first + (size_t)s * split_stride)) : make_float2(0.f, 0.f);
    float2 acc = v[0];
#pragma unroll
    for (int s = 1; s < kMaxSplitK; ++s) { acc.x += v[s].x; acc.y += v[s].y; }
    return acc;
}
__device__ __forceinline__ float4 sum_splits4(const float4* __restrict__ first, size_t split_stride4, int n_split) {
    float4 v[kMaxSplitK];
#pragma unroll
    for (int s = 0; s < kMaxSplitK; ++s) v[s] = s < n_split ? __ldcg(first + (size_t)s * split_stride4) : make_float4(0.f, 0.f, 0.f, 0.f);
    float4 acc = v[0];
#pragma unroll
    for (int s = 1; s < kMaxSplitK; ++s) { acc.x += v[s].x; acc.y += v[s].y; acc.z += v[s].z; acc.w += v[s].w; }
    return acc;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Partial result of the temperature-scaled softmax of Eq. 2 over a slice of the vocabulary:
// m = largest raw logit, idx = its (lowest) index, s = sum exp((z - m) / T).
struct SoftTriple {
    float m;
    int idx;
    float s;
};
__device__ __forceinline__ SoftTriple soft_empty() { return SoftTriple{-INFINITY, 0x7fffffff, 0.f}; }
__device__ __forceinline__ SoftTriple soft_merge(SoftTriple a, SoftTriple b, float inv_t) {
    // larger logit wins; equal logits: lower index wins
    bool a_wins = (a.m > b.m) || (a.m == b.m && a.idx < b.idx);
    SoftTriple hi = a_wins ? a : b, lo = a_wins ? b : a;
    float s = hi.s;
    if (lo.s > 0.f) s += lo.s * expf((lo.m - hi.m) * inv_t);
    return SoftTriple{hi.m, hi.idx, s};
}
__device__ __forceinline__ void soft_push(SoftTriple& t, float z, int idx, float inv_t) {
    if (z > t.m) {   // strictly larger: a later equal logit never replaces an earlier index
        t.s = t.s * expf((t.m - z) * inv_t) + 1.f;   // exp(-inf) = 0 handles the first element
        t.m = z;
        t.idx = idx;
    } else {
        t.s += expf((z - t.m) * inv_t);
    }
}

// Final merge of the per-CTA triples of an exit-confidence launch, run by the last CTA to arrive:
// warp w takes rows w, w + n_warps, ...; lane l folds CTAs l, l+32, ... in that order, then the
// lanes fold as a butterfly.  The tree is fixed by (n_ctas) alone, so the result is deterministic,
// and all loads of a lane are independent (no latency chain).
__device__ __forceinline__ void soft_final_merge(const SoftTriple* part, int n_ctas, int r0, int m, float inv_t,
                                                 float threshold, float* conf, int* token, int* exit_flag) {
    int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, n_warps = blockDim.x >> 5;
    for (int i = r0 + warp; i < r0 + m; i += n_warps) {
        SoftTriple t = soft_empty();
        for (int c = lane; c < n_ctas; c += 32) {
            const SoftTriple* p = part + (size_t)c * 8 + i;
            SoftTriple q{__ldcg(&p->m), __ldcg(&p->idx), __ldcg(&p->s)};
            t = soft_merge(t, q, inv_t);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            SoftTriple other;
            other.m = __shfl_xor_sync(0xffffffffu, t.m, o);
            other.idx = __shfl_xor_sync(0xffffffffu, t.idx, o);
            other.s = __shfl_xor_sync(0xffffffffu, t.s, o);
            t = soft_merge(t, other, inv_t);
        }
        if (lane == 0) {
            float c = 1.f / t.s;   // the arg-max term contributes exp(0) = 1, so max softmax = 1 / sum
            conf[i] = c;
            token[i] = t.idx;
            exit_flag[i] = c >= threshold ? 1 : 0;
        }
    }
}

// Result mirror: the kernel that produces what the host waits for (exit decision, acceptance) also copies the
// 49-word result block (results + status word) into host memory mapped into the device's address space and then
// writes a sequence number; the host polls that word instead of paying a copy and a stream synchronisation.
// Called by every thread of ONE CTA after its own writes to `res`; mirror may be null.
struct Mirror {
    int* host;            // device address of the mapped 64-word host block, or null
    const int* res;       // the device result block
    unsigned int seq;     // value for word 63
};
__device__ __forceinline__ void publish_results(const Mirror& m) {
    if (!m.host) return;
    __syncthreads();                                   // the CTA's writes to res
    if (threadIdx.x < 49) reinterpret_cast<volatile int*>(m.host)[threadIdx.x] = __ldcg(m.res + threadIdx.x);
    __threadfence_system();
    __syncthreads();
    if (threadIdx.x == 0) reinterpret_cast<volatile unsigned int*>(m.host)[63] = m.seq;
}

// ---- sampling decoding (Section 4.3, decoding strategies; Table 2) ----
// Counter-based uniform number that decides the token at sequence position `pos`: the splitmix64 output
// function of seed + (pos + 1) * golden-ratio increment, top 53 bits centred in their cell, in (0, 1).
__host__ __device__ inline unsigned long long sample_hash(unsigned long long seed, long long pos) {
    unsigned long long x = seed + 0x9E3779B97F4A7C15ull * (unsigned long long)(pos + 1);
    x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
    x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
    return x ^ (x >> 31);
}
__host__ __device__ inline double sample_uniform(unsigned long long seed, long long pos) {
    return ((double)(sample_hash(seed, pos) >> 11) + 0.5) * (1.0 / 9007199254740992.0);
}
constexpr int kSampleMaxVocab = 262144;
struct SampleArgs {
    const float* logits;       // [m][V] final logits, row r0 first
    double* e;                 // [m][V] scratch: exp((z - row max) / temperature), written in the kernel's first phase
    unsigned long long* q;     // [m][V] scratch: the same as 2^40 fixed-point integers (top-p select)
    int V, r0, m;
    double temperature;        // sampling temperature T_s > 0
    double top_p;              // nucleus mass; >= 1: the whole vocabulary
    unsigned long long seed;
    long long pos0;            // sequence position of the token that row r0 produces (row r0 + j: pos0 + j)
    int* token;                // token[r0 + j] receives the sample
    unsigned int* counter;     // one zero-initialised word; left at zero
    Mirror mirror;             // published by the CTA that finishes last; may be null
};

// ---------------------------------------------------------------------------------------------
// Launch arguments
// ---------------------------------------------------------------------------------------------
// Wide mode of the tcgen05 GEMM (prefill): blocks of 8 activation rows that ride through one launch.  16 blocks =
// 128 rows: MMA N = 256, two 256-column accumulators = all of an SM's tensor memory, one CTA per SM.
constexpr int kWideBlocks = 16;

struct GemmArgs {          // out[s][row][n] = sum_k act[row][k] * W[n][k]   for rows r0 .. r0+m-1
    const void* W[3];      // up to three matrices sharing K and the activation operand
    int n_end[3];          // cumulative row counts: matrix j owns output columns [n_end[j-1], n_end[j])
    int n_mats;
    int K;
    const void* act;       // Act<T> layout
    float* out;            // [n_split][8][n_total]
    int n_total;
    int r0, m;
    // tcgen05 kernel only, two matrices (gate, up) of equal shape: if set, nothing is written to out;
    // the kernel stores SwiGLU(gate, up) = silu(act.gate) * (act.up) as an Act<T> operand [.][n_end[0]] here
    void* swiglu_out;
    // tcgen05 kernel only: a later GEMM of the same stream that will run with swiglu_out set (its two
    // matrices, rows of each, K, activation operand).  This launch may prefetch part of those weights
    // into L2 while it waits for its predecessor.  Null = nothing announced.
    const void* next_W[2];
    int next_rows, next_K;
    const void* next_act;
    // tcgen05 kernel only, wide mode (prefill): nb = kWideBlocks blocks of 8 activation rows in one launch.  act is then
    // [nb][16][K] (block b = rows 8b .. 8b+7: high halves, low halves), out is [nb][n_split][8][n_total],
    // swiglu_out [nb][16][n_end[0]], and r0 / m count rows over all blocks.  0 or 1: one block.
    int nb;
};

struct HeadArgs {          // exit-confidence / final-head kernel
    const void* W;         // lm_head [V, K]
    int V, K;
    const void* act;       // Act<T> layout: final-RMSNorm of the hidden rows
    int r0, m;
    float inv_tau;
    float threshold;
    float* conf;           // [8]   indexed by row
    int* token;            // [8]
    int* exit_flag;        // [8]   conf >= threshold
    float* logits_dbg;     // nullable [m][V] (row r0 first)
    SoftTriple* part;      // scratch [kHeadMaxCtas][8]
    unsigned int* ticket;  // scratch counter, zero between launches (the kernel re-zeroes it)
    Mirror mirror;         // host.host = null: results stay on the device
};

struct AttnArgs {
    const float* q;        // [8][H*hd]
    const void* k_cache;   // [n_pages][page][kvd]
    const void* v_cache;
    const int* page_table;
    float* part;           // [n_chunks][8][H][hd+2]
    void* act_out;         // Act<T> [.][H*hd]
    int H, Hkv, hd, page, page_shift;
    int pos0;              // position of row 0
    int r0, m;
    int chunk;             // tokens per split (fixed per context)
    // fused variant only (RoPE, cache append and chunk merge inside the attention kernel)
    const float* qkv;      // QKV split-K partials [n_split][8][qd + 2 kvd]
    int n_split;
    const float2* rope_tab;   // nullable: cos/sin [position][hd/2] (launch_rope_table)
    unsigned int* status;     // device status word: a staging copy that never completes raises code 5 here
    double inv_freq[64];   // as in RopeArgs
    // separate kernels only: n_blocks > 1 runs that many blocks of 8 rows in one launch (grid.z = block); block b
    // takes rows 8b .. 8b+7 of q ([8 n_blocks][H*hd]), its own partials (part + b * part_block_stride), its own 16
    // operand rows of act_out, and sits at positions pos0 + 8b ..; r0 must be 0 and m = 8
    int n_blocks = 0;
    size_t part_block_stride = 0;
    // separate kernels only: first position that the RoPE/append launch preceding this one wrote (-1: pos0 + r0).
    // K/V rows below it belong to earlier steps and may be fetched before the grid-dependency wait.
    int pos_pred0 = -1;
    // grouped-query models: the query heads of a KV head spread over gsplit CTAs (1, 2 or 4, a divisor of H / Hkv;
    // grid.x = Hkv * gsplit), each staging the KV head's rows for itself.  Set by the launchers.
    int gsplit = 1;
};

struct RopeArgs {
    const float* qkv;      // partials [block][n_split][8][qd + 2 kvd]; block = row / 8 (one block unless m > 8)
    int n_split;
    float* q;              // [m][qd]
    void* k_cache;
    void* v_cache;
    const int* page_table;
    int H, Hkv, hd, page, page_shift;
    int pos0, r0, m;
    float rope_base;
    const float2* rope_tab;   // nullable: cos/sin [position][hd/2] (launch_rope_table)
    double inv_freq[64];   // base^(-2i/hd), i < hd/2, computed on the host in fp64
};

// ---- launchers (kernels_small.cu) ----
template <typename T> void launch_embed(cudaStream_t st, const T* embed, int d, const int* toks_dev, int tok_scalar,
                                        int row0, int m, float* h);
template <typename T> void launch_resid_norm(cudaStream_t st, float* h, const float* part, int n_split, int d,
                                             const T* gain, float eps, void* act, int r0, int m,
                                             unsigned int* clear16 = nullptr, const T* gain2 = nullptr, void* act2 = nullptr);
template <typename T> void launch_rope_append(cudaStream_t st, const RopeArgs& a);
// cos/sin of pos * inv_freq[i] for pos < n_pos, i < half, as [pos][half]
void launch_rope_table(cudaStream_t st, float2* tab, int n_pos, int half, const double* inv_freq);
// false: the shape is not covered (too many (row, query head) pairs per KV head for the shared memory of an SM); nothing launched
template <typename T> bool launch_attention(cudaStream_t st, const AttnArgs& a);
// RoPE + cache append + attention + chunk merge in one launch (a.qkv, a.n_split, a.inv_freq set; a.q unused).
// Returns false without launching when the shape is not covered (more than 8 chunks of 128 positions, or the
// device cannot co-schedule the cluster): the caller then runs launch_rope_append + launch_attention.
template <typename T> bool launch_attention_fused(cudaStream_t st, const AttnArgs& a);
// Contexts of any length (a.qkv, a.n_split, a.inv_freq set; a.q unused): the chunk kernel with RoPE and cache append
// in its front end, then the chunk merge: two launches.  Same results, bit for bit, as launch_rope_append +
// launch_attention.  Returns false without launching if the shape is not covered.
template <typename T> bool launch_attention_front(cudaStream_t st, const AttnArgs& a);
template <typename T> void launch_attention_combine(cudaStream_t st, const AttnArgs& a);
// Tiled causal attention of a wide prefill pass on the tensor cores (attn_prefill.cu; bf16 caches, head_dim 64 or 128):
// q [M][H * hd] fp32 rotated queries of the rows at positions pos0 .., whose K/V rows are in the cache already;
// act_out: the output projection's operand in the block-major layout of the wide GEMMs.  false: shape not covered.
bool launch_attention_prefill(cudaStream_t st, const float* q, const void* k_cache, const void* v_cache, const int* page_table,
                              void* act_out, int H, int Hkv, int hd, int page, int page_shift, int pos0, int M);
template <typename T> void launch_swiglu(cudaStream_t st, const float* part, int n_split, int F, void* act, int r0, int m);
void launch_accept(cudaStream_t st, const int* g, const int* drafts8, int w, int max_emit, int* result, const Mirror& mirror);
bool launch_sample(cudaStream_t st, const SampleArgs& a);   // false: the cluster launch was refused
void launch_init_pages(cudaStream_t st, int* page_table, int n_pages);

// ---- launchers (gemm_simt.cu) ----
template <typename T> void launch_gemm_simt(cudaStream_t st, const GemmArgs& a);
template <typename T> void launch_head_simt(cudaStream_t st, const HeadArgs& a, int n_ctas);

}  // namespace sb
