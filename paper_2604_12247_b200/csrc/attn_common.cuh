// Arithmetic shared by the attention kernels (one-launch cluster kernel, separate chunk kernel, streaming kernel
// for long contexts, chunk merge).  Every kernel computes a (row, query head) pair's attention the same way:
//
//   32-position block : a position's score = (fmaf chain over the even channels, in order) + (fmaf chain over the odd
//                       channels, in order); block maximum and sum of exp(score - maximum) by warp butterflies;
//                       out = sum_t p_t V_t by one fmaf chain per channel over the positions in order
//   128-position chunk: its four blocks merged at once: M = max m_j, L = sum_j l_j f_j, O = sum_j o_j f_j with
//                       f_j = exp(m_j - M), in block order
//   8-chunk group     : the chunks folded one after the other, in chunk order
//   whole context     : the groups folded one after the other, in group order;  out = O / L
//
// The roundings below are explicit (no contraction left to the compiler) so that the kernels agree bit for bit and a
// row's result depends on its own position only, never on the rows that ride along or on the launch that computes it.
#pragma once
#include "sb_internal.cuh"

namespace sb {

constexpr int kPosWarps = 4;                  // 32-position blocks per chunk
constexpr int kAttnChunk = 128;               // positions per chunk
constexpr int kChunkGroup = 8;                // chunks per group of the two-level fold
constexpr unsigned long long kStageWaitCycles = 2000000000ull;   // bound of the wait for staging copies (~1 s)

template <typename T> __device__ __forceinline__ void unpack16(const uint4& u, float (&f)[16 / sizeof(T)]);
template <> __device__ __forceinline__ void unpack16<float>(const uint4& u, float (&f)[4]) {
    f[0] = __uint_as_float(u.x); f[1] = __uint_as_float(u.y); f[2] = __uint_as_float(u.z); f[3] = __uint_as_float(u.w);
}
template <> __device__ __forceinline__ void unpack16<__nv_bfloat16>(const uint4& u, float (&f)[8]) {
    const uint32_t r[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        f[2 * j] = __uint_as_float(r[j] << 16);
        f[2 * j + 1] = __uint_as_float(r[j] & 0xffff0000u);
    }
}
// E consecutive channels (E = 1, 2 or 4) of a staged V row as floats; p is E * sizeof(T)-byte aligned
template <typename T, int E> __device__ __forceinline__ void load_channels(const unsigned char* p, float (&f)[E]);
template <> __device__ __forceinline__ void load_channels<float, 1>(const unsigned char* p, float (&f)[1]) { f[0] = *reinterpret_cast<const float*>(p); }
template <> __device__ __forceinline__ void load_channels<float, 2>(const unsigned char* p, float (&f)[2]) {
    const float2 v = *reinterpret_cast<const float2*>(p); f[0] = v.x; f[1] = v.y;
}
template <> __device__ __forceinline__ void load_channels<float, 4>(const unsigned char* p, float (&f)[4]) {
    const float4 v = *reinterpret_cast<const float4*>(p); f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w;
}
template <> __device__ __forceinline__ void load_channels<__nv_bfloat16, 1>(const unsigned char* p, float (&f)[1]) {
    f[0] = __uint_as_float((uint32_t)*reinterpret_cast<const unsigned short*>(p) << 16);
}
template <> __device__ __forceinline__ void load_channels<__nv_bfloat16, 2>(const unsigned char* p, float (&f)[2]) {
    const uint32_t r = *reinterpret_cast<const uint32_t*>(p);
    f[0] = __uint_as_float(r << 16); f[1] = __uint_as_float(r & 0xffff0000u);
}
template <> __device__ __forceinline__ void load_channels<__nv_bfloat16, 4>(const unsigned char* p, float (&f)[4]) {
    const uint2 r = *reinterpret_cast<const uint2*>(p);
    f[0] = __uint_as_float(r.x << 16); f[1] = __uint_as_float(r.x & 0xffff0000u);
    f[2] = __uint_as_float(r.y << 16); f[3] = __uint_as_float(r.y & 0xffff0000u);
}

// ---- rotary embedding: rotate-half pairing (i, i + hd/2), angle = pos * base^(-2i/hd) ----
// cos and sin of the angle pos * inv_freq[i]
__device__ __forceinline__ float2 rope_cos_sin(const double* inv_freq, int pos, int i) {
    // the angle is formed and reduced to [-pi, pi] in fp64 (exact for every position), then
    // the fp32 sincos sees a small argument
    double ang = (double)pos * inv_freq[i];
    ang -= 6.283185307179586476925 * rint(ang * 0.15915494309189533577);
    float s, c;
    sincosf((float)ang, &s, &c);
    return make_float2(c, s);
}
// cos/sin of the angle of rotation pair i at position pos; tab (nullable) = rope_cos_sin tabulated as
// [position][hd/2] by k_rope_table: the same values, one load instead of the math
__device__ __forceinline__ float2 rope_fetch(const double* inv_freq, const float2* __restrict__ tab, int half, int pos, int i) {
    return tab ? __ldg(tab + (size_t)pos * half + i) : rope_cos_sin(inv_freq, pos, i);
}
// rotate the pair (x0, x1) = elements (i, i + hd/2) of a head
__device__ __forceinline__ void rope_apply(float2 cs, float& x0, float& x1) {
    // explicit roundings: the compiler must not contract these into fused multiply-adds differently at
    // different call sites (the separate and the fused kernels have to agree bit for bit)
    float y0 = __fsub_rn(__fmul_rn(x0, cs.x), __fmul_rn(x1, cs.y)), y1 = __fadd_rn(__fmul_rn(x1, cs.x), __fmul_rn(x0, cs.y));
    x0 = y0;
    x1 = y1;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// acc[e] = fma(p, v[e], acc[e]) for a lane's E channels: one rounding per channel, two channels per instruction
// (fma.rn.f32x2 is two independent IEEE fused multiply-adds) where E is even
template <int E> __device__ __forceinline__ void fma_channels(float p, const float (&v)[E], float (&acc)[E]) {
    if constexpr (E % 2 == 0) {
        const float2 pp = make_float2(p, p);
#pragma unroll
        for (int e = 0; e < E; e += 2) {
            const float2 r = __ffma2_rn(pp, make_float2(v[e], v[e + 1]), make_float2(acc[e], acc[e + 1]));
            acc[e] = r.x;
            acc[e + 1] = r.y;
        }
    } else {
#pragma unroll
        for (int e = 0; e < E; ++e) acc[e] = fmaf(p, v[e], acc[e]);
    }
}

// One step of a position's score: channels c .. c+3 of q and K enter the accumulator, whose halves are the running sums
// over the even and over the odd channels (each a fused-multiply-add chain in channel order, advanced together by packed
// instructions: neither operand has to be duplicated, and the dependent chain is half as long as one sum over all
// channels would be).  attn_score_finish adds the two halves.
__device__ __forceinline__ void attn_score_step(const float4& q, float k0, float k1, float k2, float k3, float2& acc) {
    acc = __ffma2_rn(make_float2(q.x, q.y), make_float2(k0, k1), acc);
    acc = __ffma2_rn(make_float2(q.z, q.w), make_float2(k2, k3), acc);
}
__device__ __forceinline__ float attn_score_finish(const float2& acc) { return __fadd_rn(acc.x, acc.y); }

// x / d for a small non-negative x and the query-head group size d: a shift where d is a power of two (the usual
// group sizes; a run-time integer division costs about twenty instructions, and the kernels divide once per work item)
struct GroupDiv {
    int d, sh;
    __device__ explicit GroupDiv(int d_) : d(d_), sh(-1) {
        if ((d_ & (d_ - 1)) == 0)
            for (sh = 0; (1 << sh) < d_; ++sh) {}
    }
    __device__ __forceinline__ int operator()(int x) const { return sh >= 0 ? x >> sh : (int)((unsigned)x / (unsigned)d); }
};

// N (1 or 2) consecutive values rounded to the storage type and stored at p (N * sizeof(T)-byte aligned), as one store
template <typename T, int N> __device__ __forceinline__ void store_run(T* p, const float (&v)[N]);
template <> __device__ __forceinline__ void store_run<float, 1>(float* p, const float (&v)[1]) { p[0] = v[0]; }
template <> __device__ __forceinline__ void store_run<float, 2>(float* p, const float (&v)[2]) {
    *reinterpret_cast<float2*>(p) = make_float2(v[0], v[1]);
}
template <> __device__ __forceinline__ void store_run<__nv_bfloat16, 1>(__nv_bfloat16* p, const float (&v)[1]) { p[0] = from_f32<__nv_bfloat16>(v[0]); }
template <> __device__ __forceinline__ void store_run<__nv_bfloat16, 2>(__nv_bfloat16* p, const float (&v)[2]) {
    __nv_bfloat162 r;
    r.x = from_f32<__nv_bfloat16>(v[0]);
    r.y = from_f32<__nv_bfloat16>(v[1]);
    *reinterpret_cast<__nv_bfloat162*>(p) = r;
}

// 1 / sqrt(head_dim) as every kernel forms it
__device__ __forceinline__ float attn_score_scale(int hd) { return rsqrtf((float)hd); }

// Softmax pieces of one 32-position block for one pair: lane = position.  `on`: the position is visible to the
// pair's row (causal mask).  Returns this lane's probability relative to the block maximum; m = block maximum
// (-inf if no position is visible), l = sum of the probabilities.
__device__ __forceinline__ float attn_block_softmax(float score, float scale, bool on, float& m_out, float& l_out) {
    const float s = on ? __fmul_rn(score, scale) : -INFINITY;
    float m = s;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    float pt = 0.f;
    m_out = -INFINITY;
    l_out = 0.f;
    if (m > -INFINITY) {
        pt = on ? expf(__fsub_rn(s, m)) : 0.f;
        m_out = m;
        l_out = warp_sum(pt);
    }
    return pt;
}
// weight of a block partial with maximum m inside a chunk whose maximum is M
__device__ __forceinline__ float attn_block_weight(float m, float M) { return expf(__fsub_rn(m, M)); }
// acc + x * f in one rounding (the chunk's L and O sums)
__device__ __forceinline__ float attn_weighted_add(float acc, float x, float f) { return __fmaf_rn(x, f, acc); }
// One step of the in-order fold: the running (M, L) takes in a partial (mc, lc); f0 and f1 are the factors by which the
// running and the incoming out vectors are scaled (attn_fold_out).  Call only for mc > -inf.
__device__ __forceinline__ void attn_fold(float& M, float& L, float mc, float lc, float& f0, float& f1) {
    const float nm = fmaxf(M, mc);
    f0 = expf(__fsub_rn(M, nm));
    f1 = expf(__fsub_rn(mc, nm));
    L = __fmaf_rn(L, f0, __fmul_rn(lc, f1));
    M = nm;
}
__device__ __forceinline__ float attn_fold_out(float O, float oc, float f0, float f1) { return __fmaf_rn(O, f0, __fmul_rn(oc, f1)); }
__device__ __forceinline__ float attn_finish(float O, float L) { return __fdiv_rn(O, L); }

}  // namespace sb
