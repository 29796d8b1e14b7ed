// Small kernels of the layer pass: embedding gather, residual + RMSNorm, RoPE + KV append,
// decode attention over the paged KV cache (split-KV, warp-shuffle reductions), SwiGLU,
// greedy acceptance.  All of them are deterministic and row-invariant: what they compute for one
// row never depends on which other rows ride along in the same launch.
#include "sb_internal.cuh"

namespace sb {

bool g_use_pdl = true;

// ------------------------------------------------------------------------------------------------
// h[row0 + i] = embed[token_i]
// ------------------------------------------------------------------------------------------------
template <typename T>
__global__ void k_embed(const T* __restrict__ embed, int d, const int* __restrict__ toks, int tok_scalar, int row0,
                        float* __restrict__ h) {
    pdl_trigger();
    pdl_wait();
    int i = blockIdx.x;
    int tok = toks ? toks[i] : tok_scalar;
    const T* src = embed + (size_t)tok * d;
    float* dst = h + (size_t)(row0 + i) * d;
    for (int k = threadIdx.x; k < d; k += blockDim.x) dst[k] = to_f32(src[k]);
}
template <typename T>
void launch_embed(cudaStream_t st, const T* embed, int d, const int* toks_dev, int tok_scalar, int row0, int m, float* h) {
    launch_k(k_embed<T>, dim3(m), dim3(256), 0, st, embed, d, toks_dev, tok_scalar, row0, h);
}

// ------------------------------------------------------------------------------------------------
// h[row] += sum_s part[s][row][:]   (if part != null; split-K partials are summed in split order)
// act[row] = h[row] / sqrt(mean(h[row]^2) + eps) * gain      (if gain != null)
// One CTA per row; the reduction order is fixed by the thread layout only.
// ------------------------------------------------------------------------------------------------
constexpr int kNormThreads = 1024;
constexpr int kNormVec = 2;   // float4 per thread: rows up to 1024 * 2 * 4 = 8192 wide
template <typename T>
__global__ void __launch_bounds__(kNormThreads) k_resid_norm(float* __restrict__ h, const float* __restrict__ part,
                                                            int n_split, int d, const T* __restrict__ gain, float eps,
                                                            void* __restrict__ act, int r0) {
    __shared__ float red[kNormThreads / 32];
    pdl_trigger();
    pdl_wait();
    int row = r0 + blockIdx.x;
    float4* hr = reinterpret_cast<float4*>(h + (size_t)row * d);
    const int nv = d >> 2;
    float4 v[kNormVec];
    float ss = 0.f;
    // every load of a thread is independent: the hidden row and all partials are in flight at once
#pragma unroll
    for (int j = 0; j < kNormVec; ++j) {
        int k4 = threadIdx.x + j * kNormThreads;
        if (k4 < nv) {
            v[j] = hr[k4];
            if (part) {
                for (int s = 0; s < n_split; ++s) {   // summed in split order
                    float4 p = __ldcg(reinterpret_cast<const float4*>(part + ((size_t)s * kMaxW + row) * d) + k4);
                    v[j].x += p.x; v[j].y += p.y; v[j].z += p.z; v[j].w += p.w;
                }
                hr[k4] = v[j];
            }
            ss += v[j].x * v[j].x + v[j].y * v[j].y + v[j].z * v[j].z + v[j].w * v[j].w;
        }
    }
    if (!gain) return;
    ss = warp_sum(ss);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
    __syncthreads();
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < kNormThreads / 32; ++w) tot += red[w];
    float inv = rsqrtf(tot / (float)d + eps);
    using A = Act<T>;
    typename A::type* a = reinterpret_cast<typename A::type*>(act);
#pragma unroll
    for (int j = 0; j < kNormVec; ++j) {
        int k4 = threadIdx.x + j * kNormThreads;
        if (k4 < nv) {
            int k = k4 << 2;
            A::store(a, row, k, d, v[j].x * inv * to_f32(gain[k]));
            A::store(a, row, k + 1, d, v[j].y * inv * to_f32(gain[k + 1]));
            A::store(a, row, k + 2, d, v[j].z * inv * to_f32(gain[k + 2]));
            A::store(a, row, k + 3, d, v[j].w * inv * to_f32(gain[k + 3]));
        }
    }
}
template <typename T>
void launch_resid_norm(cudaStream_t st, float* h, const float* part, int n_split, int d, const T* gain, float eps,
                       void* act, int r0, int m) {
    launch_k(k_resid_norm<T>, dim3(m), dim3(kNormThreads), 0, st, h, part, n_split, d, gain, eps, act, r0);
}

// ------------------------------------------------------------------------------------------------
// Sum the QKV split-K partials, rotate q and k (rotate-half pairing, angle = pos * base^(-2i/hd)),
// write q (fp32) and append k, v to the paged cache in the storage dtype.
// grid = (H + 2 Hkv, m), block = hd/2 threads (one rotation pair each).
// ------------------------------------------------------------------------------------------------
template <typename T>
__global__ void k_rope_append(RopeArgs a) {
    pdl_trigger();
    pdl_wait();
    int head = blockIdx.x;
    int row = a.r0 + blockIdx.y;
    int pos = a.pos0 + row;
    int half = a.hd >> 1;
    int i = threadIdx.x;
    int qd = a.H * a.hd, kvd = a.Hkv * a.hd, ntot = qd + 2 * kvd;
    int col = head * a.hd;   // q heads, then k heads, then v heads are contiguous in the GEMM output
    float x0 = 0.f, x1 = 0.f;
    for (int s = 0; s < a.n_split; ++s) {
        const float* p = a.qkv + ((size_t)s * kMaxW + row) * ntot + col;
        x0 += p[i];
        x1 += p[i + half];
    }
    bool is_v = head >= a.H + a.Hkv;
    if (!is_v) {
        // the angle is formed and reduced to [-pi, pi] in fp64 (exact for every position), then
        // the fp32 sincos sees a small argument
        double ang = (double)pos * a.inv_freq[i];
        ang -= 6.283185307179586476925 * rint(ang * 0.15915494309189533577);
        float s, c;
        sincosf((float)ang, &s, &c);
        float y0 = x0 * c - x1 * s, y1 = x1 * c + x0 * s;
        x0 = y0;
        x1 = y1;
    }
    if (head < a.H) {
        float* q = a.q + (size_t)row * qd + col;
        q[i] = x0;
        q[i + half] = x1;
    } else {
        int kvh = is_v ? head - a.H - a.Hkv : head - a.H;
        T* cache = reinterpret_cast<T*>(is_v ? a.v_cache : a.k_cache);
        int page = a.page_table[pos >> a.page_shift];
        T* dst = cache + ((size_t)page * a.page + (pos & (a.page - 1))) * kvd + kvh * a.hd;
        dst[i] = from_f32<T>(x0);
        dst[i + half] = from_f32<T>(x1);
    }
}
template <typename T> void launch_rope_append(cudaStream_t st, const RopeArgs& a) {
    dim3 grid(a.H + 2 * a.Hkv, a.m);
    launch_k(k_rope_append<T>, grid, dim3(a.hd / 2), 0, st, a);
}

// ------------------------------------------------------------------------------------------------
// Decode attention, split over the KV length in chunks whose boundaries depend on absolute
// positions only.  grid = (H, n_chunks); 4 warps; warp v of a CTA takes tokens base+v, base+v+4, ...
// A lane owns hd/32 contiguous channels; q.k is reduced with warp shuffles; the running
// (max, sum, out) of every row lives in registers.  Per-(chunk,row,head) partials go to scratch
// and k_attn_combine merges them in chunk order.
// ------------------------------------------------------------------------------------------------
constexpr int kAttnWarps = 4;
template <typename T, int E>   // E = hd / 32
__global__ void __launch_bounds__(kAttnWarps * 32) k_attn_partial(AttnArgs a) {
    constexpr int HD = E * 32;
    __shared__ float q_s[kMaxW][HD];
    __shared__ float mrg[kAttnWarps][kMaxW][HD + 2];
    pdl_trigger();
    pdl_wait();
    int hq = blockIdx.x, c = blockIdx.y;
    int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int kvh = hq / (a.H / a.Hkv);
    int kvd = a.Hkv * HD, qd = a.H * HD;
    int t_begin = c * a.chunk;
    int pos_last = a.pos0 + a.r0 + a.m - 1;
    int t_end = min(t_begin + a.chunk, pos_last + 1);
    for (int idx = threadIdx.x; idx < a.m * HD; idx += blockDim.x) {
        int i = idx / HD, e = idx - i * HD;
        q_s[i][e] = a.q[(size_t)(a.r0 + i) * qd + hq * HD + e];
    }
    __syncthreads();
    const float scale = rsqrtf((float)HD);
    float mx[kMaxW], l[kMaxW], o[kMaxW][E];
#pragma unroll
    for (int i = 0; i < kMaxW; ++i) {
        mx[i] = -INFINITY;
        l[i] = 0.f;
#pragma unroll
        for (int e = 0; e < E; ++e) o[i][e] = 0.f;
    }
    const T* kc = reinterpret_cast<const T*>(a.k_cache);
    const T* vc = reinterpret_cast<const T*>(a.v_cache);
    for (int t = t_begin + warp; t < t_end; t += kAttnWarps) {
        int page = a.page_table[t >> a.page_shift];
        size_t off = ((size_t)page * a.page + (t & (a.page - 1))) * kvd + kvh * HD + lane * E;
        float kf[E], vf[E];
#pragma unroll
        for (int e = 0; e < E; ++e) {
            kf[e] = to_f32(kc[off + e]);
            vf[e] = to_f32(vc[off + e]);
        }
#pragma unroll
        for (int i = 0; i < kMaxW; ++i) {
            if (i < a.m && t <= a.pos0 + a.r0 + i) {   // causal: row i sees positions <= its own
                float s = 0.f;
#pragma unroll
                for (int e = 0; e < E; ++e) s += q_s[i][lane * E + e] * kf[e];
                s = warp_sum(s) * scale;
                float nm = fmaxf(mx[i], s);
                float corr = expf(mx[i] - nm);   // exp(-inf) = 0 on the first token
                float p = expf(s - nm);
                l[i] = l[i] * corr + p;
#pragma unroll
                for (int e = 0; e < E; ++e) o[i][e] = o[i][e] * corr + p * vf[e];
                mx[i] = nm;
            }
        }
    }
#pragma unroll
    for (int i = 0; i < kMaxW; ++i) {
        if (i < a.m) {
#pragma unroll
            for (int e = 0; e < E; ++e) mrg[warp][i][lane * E + e] = o[i][e];
            if (lane == 0) {
                mrg[warp][i][HD] = mx[i];
                mrg[warp][i][HD + 1] = l[i];
            }
        }
    }
    __syncthreads();
    // merge the four warps in warp order; thread -> (row, channel)
    for (int idx = threadIdx.x; idx < a.m * HD; idx += blockDim.x) {
        int i = idx / HD, e = idx - i * HD;
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < kAttnWarps; ++w) M = fmaxf(M, mrg[w][i][HD]);
        float L = 0.f, O = 0.f;
        if (M > -INFINITY) {
#pragma unroll
            for (int w = 0; w < kAttnWarps; ++w) {
                float mw = mrg[w][i][HD];
                if (mw > -INFINITY) {
                    float f = expf(mw - M);
                    L += mrg[w][i][HD + 1] * f;
                    O += mrg[w][i][e] * f;
                }
            }
        }
        float* dst = a.part + (((size_t)c * kMaxW + (a.r0 + i)) * a.H + hq) * (HD + 2);
        dst[e] = O;
        if (e == 0) {
            dst[HD] = M;
            dst[HD + 1] = L;
        }
    }
}

// grid = (H, m), block = hd: merge the chunk partials of one (row, head) in chunk order.
template <typename T>
__global__ void k_attn_combine(AttnArgs a) {
    pdl_trigger();
    pdl_wait();
    int hq = blockIdx.x, row = a.r0 + blockIdx.y, e = threadIdx.x;
    int hd = a.hd;
    int n_chunks = (a.pos0 + row) / a.chunk + 1;   // chunks that hold positions <= this row's own
    float M = -INFINITY, L = 0.f, O = 0.f;
    for (int c = 0; c < n_chunks; ++c) {
        const float* src = a.part + (((size_t)c * kMaxW + row) * a.H + hq) * (hd + 2);
        float mc = src[hd];
        if (mc == -INFINITY) continue;
        float nm = fmaxf(M, mc);
        float f0 = expf(M - nm), f1 = expf(mc - nm);
        L = L * f0 + src[hd + 1] * f1;
        O = O * f0 + src[e] * f1;
        M = nm;
    }
    using A = Act<T>;
    A::store(reinterpret_cast<typename A::type*>(a.act_out), row, hq * hd + e, a.H * hd, O / L);
}

template <typename T> void launch_attention(cudaStream_t st, const AttnArgs& a) {
    int n_chunks = (a.pos0 + a.r0 + a.m - 1) / a.chunk + 1;
    dim3 grid(a.H, n_chunks);
    switch (a.hd) {
        case 32: launch_k(k_attn_partial<T, 1>, grid, dim3(kAttnWarps * 32), 0, st, a); break;
        case 64: launch_k(k_attn_partial<T, 2>, grid, dim3(kAttnWarps * 32), 0, st, a); break;
        default: launch_k(k_attn_partial<T, 4>, grid, dim3(kAttnWarps * 32), 0, st, a); break;
    }
    launch_k(k_attn_combine<T>, dim3(a.H, a.m), dim3(a.hd), 0, st, a);
}

// ------------------------------------------------------------------------------------------------
// act[row][f] = silu(sum_s gate) * (sum_s up);  partials are [s][8][2F] with gate | up columns
// ------------------------------------------------------------------------------------------------
template <typename T>
__global__ void k_swiglu(const float* __restrict__ part, int n_split, int F, void* __restrict__ act, int r0) {
    pdl_trigger();
    pdl_wait();
    int row = r0 + blockIdx.y;
    int f = blockIdx.x * blockDim.x + threadIdx.x;
    if (f >= F) return;
    float g = 0.f, u = 0.f;
    for (int s = 0; s < n_split; ++s) {
        const float* p = part + ((size_t)s * kMaxW + row) * (2 * (size_t)F);
        g += p[f];
        u += p[F + f];
    }
    float v = g / (1.f + expf(-g)) * u;
    using A = Act<T>;
    A::store(reinterpret_cast<typename A::type*>(act), row, f, F, v);
}
template <typename T> void launch_swiglu(cudaStream_t st, const float* part, int n_split, int F, void* act, int r0, int m) {
    launch_k(k_swiglu<T>, dim3((F + 255) / 256, m), dim3(256), 0, st, part, n_split, F, act, r0);
}

// ------------------------------------------------------------------------------------------------
// Greedy acceptance: the longest prefix of drafts equal to the full model's tokens, then the
// model's own token.  result = {n_emit, n_accepted_drafts, g[0..7]}
// ------------------------------------------------------------------------------------------------
struct Drafts8 { int v[kMaxW]; };
__global__ void k_accept(const int* __restrict__ g, Drafts8 drafts, int w, int max_emit, int* __restrict__ result) {
    pdl_trigger();
    pdl_wait();
    if (threadIdx.x != 0) return;
    int acc = 0;
    while (acc < w && drafts.v[acc] >= 0 && g[acc] == drafts.v[acc]) ++acc;
    int emit = acc < w ? acc + 1 : w;
    if (emit > max_emit) emit = max_emit;
    result[0] = emit;
    result[1] = acc;
    for (int i = 0; i < kMaxW; ++i) result[2 + i] = i < w ? g[i] : -1;
}
void launch_accept(cudaStream_t st, const int* g, const int* drafts8, int w, int max_emit, int* result) {
    Drafts8 d;
    for (int i = 0; i < kMaxW; ++i) d.v[i] = drafts8[i];
    launch_k(k_accept, dim3(1), dim3(32), 0, st, g, d, w, max_emit, result);
}

__global__ void k_init_pages(int* pt, int n) {
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) pt[i] = i;
}
void launch_init_pages(cudaStream_t st, int* page_table, int n_pages) {
    k_init_pages<<<(n_pages + 255) / 256, 256, 0, st>>>(page_table, n_pages);
}

// explicit instantiations
#define SB_INST(T)                                                                                                  \
    template void launch_embed<T>(cudaStream_t, const T*, int, const int*, int, int, int, float*);                  \
    template void launch_resid_norm<T>(cudaStream_t, float*, const float*, int, int, const T*, float, void*, int, int); \
    template void launch_rope_append<T>(cudaStream_t, const RopeArgs&);                                             \
    template void launch_attention<T>(cudaStream_t, const AttnArgs&);                                               \
    template void launch_swiglu<T>(cudaStream_t, const float*, int, int, void*, int, int);
SB_INST(float)
SB_INST(__nv_bfloat16)

}  // namespace sb
