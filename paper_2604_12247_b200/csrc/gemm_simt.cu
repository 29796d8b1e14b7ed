// CUDA-core weight-streaming kernels: the skinny GEMM  out[row][n] = sum_k act[row][k] W[n][k]
// for up to 8 rows, and the exit-confidence kernel (LM-head GEMV fused with the online
// temperature-scaled softmax max / argmax of Eq. 2).  One warp per output row, 128-bit coalesced
// weight loads, fp32 accumulation.  These cover every dtype (fp32 models never use tensor cores:
// tf32 would break their 1e-4 logit tolerance) and are the reference path for the tcgen05 kernels.
#include "sb_internal.cuh"

namespace sb {

// eight consecutive weights of a row as floats
__device__ __forceinline__ void load8(const float* p, float (&w)[8]) {
    float4 a = __ldg(reinterpret_cast<const float4*>(p));
    float4 b = __ldg(reinterpret_cast<const float4*>(p) + 1);
    w[0] = a.x; w[1] = a.y; w[2] = a.z; w[3] = a.w; w[4] = b.x; w[5] = b.y; w[6] = b.z; w[7] = b.w;
}
__device__ __forceinline__ void load8(const __nv_bfloat16* p, float (&w)[8]) {
    uint4 u = __ldg(reinterpret_cast<const uint4*>(p));
    const uint32_t r[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        w[2 * j] = __uint_as_float(r[j] << 16);
        w[2 * j + 1] = __uint_as_float(r[j] & 0xffff0000u);
    }
}
// eight consecutive activations of row `row` as floats
__device__ __forceinline__ void load_act8(const float* a, int row, int k, int K, float (&x)[8]) {
    load8(a + (size_t)row * K + k, x);
}
__device__ __forceinline__ void load_act8(const __nv_bfloat16* a, int row, int k, int K, float (&x)[8]) {
    float lo[8];
    load8(a + (size_t)row * K + k, x);
    load8(a + (size_t)(row + 8) * K + k, lo);
#pragma unroll
    for (int j = 0; j < 8; ++j) x[j] += lo[j];
}

// dot products of one weight row with the activation rows r0 .. r0+m-1 (all lanes get the sums)
template <typename T>
__device__ __forceinline__ void row_dots(const T* __restrict__ wrow, const typename Act<T>::type* __restrict__ act, int K,
                                         int r0, int m, int lane, float (&acc)[kMaxW]) {
#pragma unroll
    for (int i = 0; i < kMaxW; ++i) acc[i] = 0.f;
    for (int k = lane * 8; k < K; k += 256) {
        float w[8];
        load8(wrow + k, w);
#pragma unroll
        for (int i = 0; i < kMaxW; ++i) {
            if (i >= r0 && i < r0 + m) {
                float x[8];
                load_act8(act, i, k, K, x);
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[i] = fmaf(w[j], x[j], acc[i]);
            }
        }
    }
#pragma unroll
    for (int i = 0; i < kMaxW; ++i)
        if (i >= r0 && i < r0 + m) acc[i] = warp_sum(acc[i]);
}

template <typename T>
__global__ void __launch_bounds__(256) k_gemm_simt(GemmArgs a) {
    using AT = typename Act<T>::type;
    pdl_trigger();
    pdl_wait();
    const AT* act = reinterpret_cast<const AT*>(a.act);
    int lane = threadIdx.x & 31;
    int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    int n_warps = (gridDim.x * blockDim.x) >> 5;
    for (int n = warp; n < a.n_total; n += n_warps) {
        int j = 0, base = 0;
        while (n >= a.n_end[j]) base = a.n_end[j++];
        const T* wrow = reinterpret_cast<const T*>(a.W[j]) + (size_t)(n - base) * a.K;
        float acc[kMaxW];
        row_dots<T>(wrow, act, a.K, a.r0, a.m, lane, acc);
        if (lane == 0) {
#pragma unroll
            for (int i = 0; i < kMaxW; ++i)
                if (i >= a.r0 && i < a.r0 + a.m) a.out[(size_t)i * a.n_total + n] = acc[i];
        }
    }
}
template <typename T> void launch_gemm_simt(cudaStream_t st, const GemmArgs& a) {
    int ctas = min((a.n_total + 7) / 8, 148 * 8);
    launch_k(k_gemm_simt<T>, dim3(ctas), dim3(256), 0, st, a);
}

// ------------------------------------------------------------------------------------------------
// Exit-confidence kernel (CUDA-core variant).  Every warp walks vocabulary rows v = warp, warp +
// n_warps, ... and keeps, per activation row, the running triple (max logit, its index, sum of
// exp((z - max)/T)).  Warps of a CTA are merged in warp order, CTAs in CTA order by the last CTA
// to arrive (a wait-free ticket), so the result is deterministic.  conf = 1 / sum.
// ------------------------------------------------------------------------------------------------
constexpr int kHeadWarps = 8;
template <typename T>
__global__ void __launch_bounds__(kHeadWarps * 32) k_head_simt(HeadArgs a) {
    using AT = typename Act<T>::type;
    __shared__ SoftTriple cta_part[kHeadWarps][kMaxW];
    __shared__ bool is_last;
    pdl_trigger();
    pdl_wait();
    const AT* act = reinterpret_cast<const AT*>(a.act);
    int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    int warp = blockIdx.x * kHeadWarps + wib;
    int n_warps = gridDim.x * kHeadWarps;
    SoftTriple tr[kMaxW];
#pragma unroll
    for (int i = 0; i < kMaxW; ++i) tr[i] = soft_empty();
    for (int v = warp; v < a.V; v += n_warps) {
        const T* wrow = reinterpret_cast<const T*>(a.W) + (size_t)v * a.K;
        float acc[kMaxW];
        row_dots<T>(wrow, act, a.K, a.r0, a.m, lane, acc);
#pragma unroll
        for (int i = 0; i < kMaxW; ++i) {
            if (i >= a.r0 && i < a.r0 + a.m) {
                soft_push(tr[i], acc[i], v, a.inv_tau);
                if (a.logits_dbg && lane == 0) a.logits_dbg[(size_t)(i - a.r0) * a.V + v] = acc[i];
            }
        }
    }
    if (lane == 0) {
#pragma unroll
        for (int i = 0; i < kMaxW; ++i) cta_part[wib][i] = tr[i];
    }
    __syncthreads();
    if (threadIdx.x < kMaxW) {
        int i = threadIdx.x;
        SoftTriple t = cta_part[0][i];
        for (int w = 1; w < kHeadWarps; ++w) t = soft_merge(t, cta_part[w][i], a.inv_tau);
        a.part[(size_t)blockIdx.x * kMaxW + i] = t;
        __threadfence();
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned int prev = atomicAdd(a.ticket, 1u);
        is_last = (prev == gridDim.x - 1);
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    soft_final_merge(a.part, (int)gridDim.x, a.r0, a.m, a.inv_tau, a.threshold, a.conf, a.token, a.exit_flag);
    if (threadIdx.x == 0) *a.ticket = 0u;   // ready for the next launch on this stream
    publish_results(a.mirror);
}
template <typename T> void launch_head_simt(cudaStream_t st, const HeadArgs& a, int n_ctas) {
    launch_k(k_head_simt<T>, dim3(n_ctas), dim3(kHeadWarps * 32), 0, st, a);
}

template void launch_gemm_simt<float>(cudaStream_t, const GemmArgs&);
template void launch_gemm_simt<__nv_bfloat16>(cudaStream_t, const GemmArgs&);
template void launch_head_simt<float>(cudaStream_t, const HeadArgs&, int);
template void launch_head_simt<__nv_bfloat16>(cudaStream_t, const HeadArgs&, int);

}  // namespace sb
