// Small kernels of the layer pass: embedding gather, residual + RMSNorm, RoPE + KV append,
// decode attention over the paged KV cache (split-KV, warp-shuffle reductions), SwiGLU,
// greedy acceptance.  All of them are deterministic and row-invariant: what they compute for one
// row never depends on which other rows ride along in the same launch.
#include "attn_common.cuh"
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
    // Every step of a row (a prompt block, a drafted token, an autoregressive token) starts with this kernel, and it is
    // launched WITHOUT programmatic dependent launch: it starts only after everything before it in the stream has
    // completed.  The kernels behind it may therefore rely on what earlier steps wrote (the K/V rows of earlier
    // positions) being complete even before their own grid-dependency wait returns.
    (void)launch_kcp(k_embed<T>, dim3(m), dim3(256), 0, st, 1, /*pdl=*/false, embed, d, toks_dev, tok_scalar, row0, h);
}

// ------------------------------------------------------------------------------------------------
// h[row] += sum_s part[s][row][:]   (if part != null; split-K partials are summed in split order)
// act[row] = h[row] / sqrt(mean(h[row]^2) + eps) * gain      (if gain != null)
// act2[row] = the same with gain2                             (if gain2 != null: the rows are about to be read under two
//                                                              norms, the exit test's and the next layer's)
// One CTA per row; the reduction order is fixed by the thread layout only.
// ------------------------------------------------------------------------------------------------
constexpr int kNormThreads = 1024;
constexpr int kNormVec = 2;   // float4 per thread: rows up to 1024 * 2 * 4 = 8192 wide
// kDual: a second gain and output (an instantiation of its own: the common form stays as small as it was)
template <typename T, bool kWide, bool kDual>
__global__ void __launch_bounds__(kNormThreads) k_resid_norm(float* __restrict__ h, const float* __restrict__ part,
                                                            int n_split, int d, const T* __restrict__ gain, float eps,
                                                            void* __restrict__ act, int r0, unsigned int* __restrict__ clear16,
                                                            const T* __restrict__ gain2, void* __restrict__ act2) {
    __shared__ float red[kNormThreads / 32];
    pdl_trigger();
    // the gains are weights: no kernel writes them, so they are requested before the grid-dependency wait (a layer's
    // gains were last touched a whole token ago and come from HBM)
    const int nv = d >> 2;
    float4 g4[kNormVec];
    if (gain) {
#pragma unroll
        for (int j = 0; j < kNormVec; ++j) {
            int k4 = threadIdx.x + j * kNormThreads;
            if (k4 < nv) g4[j] = load_gain4(gain, k4 << 2);
        }
    }
    float4 g4b[kNormVec];
    if (kDual) {
#pragma unroll
        for (int j = 0; j < kNormVec; ++j) {
            int k4 = threadIdx.x + j * kNormThreads;
            if (k4 < nv) g4b[j] = load_gain4(gain2, k4 << 2);
        }
    }
    pdl_wait();
    // optional: zero 16 words for the kernels that follow (the stateless calls' status word and ticket)
    if (clear16 && blockIdx.x == 0 && threadIdx.x < 16) clear16[threadIdx.x] = 0u;
    // kWide: rows beyond the first 8 (wide prefill passes) live in further blocks of 8: their split-K partials are
    // [block][split][8][d] and their operand rows [block][Act rows][d]; the hidden rows are contiguous
    const int row_all = r0 + blockIdx.x, blk = kWide ? row_all / kMaxW : 0, row = row_all - blk * kMaxW;
    float4* hr = reinterpret_cast<float4*>(h + (size_t)row_all * d);
    const float* __restrict__ part_b = part + ((size_t)blk * n_split * kMaxW + row) * d;   // this row's first partial
    float4 v[kNormVec];
    float ss = 0.f;
    // every load of a thread is independent: the hidden row, all partials and the gains are in flight at once
#pragma unroll
    for (int j = 0; j < kNormVec; ++j) {
        int k4 = threadIdx.x + j * kNormThreads;
        if (k4 < nv) {
            v[j] = hr[k4];
            if (part) {
                float4 p = sum_splits4(reinterpret_cast<const float4*>(part_b) + k4, (size_t)kMaxW * d / 4, n_split);
                v[j].x += p.x; v[j].y += p.y; v[j].z += p.z; v[j].w += p.w;
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
    typename A::type* a = reinterpret_cast<typename A::type*>(act) + (size_t)blk * A::rows * d;
#pragma unroll
    for (int j = 0; j < kNormVec; ++j) {
        int k4 = threadIdx.x + j * kNormThreads;
        if (k4 < nv)
            A::store4(a, row, k4 << 2, d, make_float4(v[j].x * inv * g4[j].x, v[j].y * inv * g4[j].y, v[j].z * inv * g4[j].z,
                                                     v[j].w * inv * g4[j].w));
    }
    if (kDual) {
        typename A::type* a2 = reinterpret_cast<typename A::type*>(act2) + (size_t)blk * A::rows * d;
#pragma unroll
        for (int j = 0; j < kNormVec; ++j) {
            int k4 = threadIdx.x + j * kNormThreads;
            if (k4 < nv)
                A::store4(a2, row, k4 << 2, d, make_float4(v[j].x * inv * g4b[j].x, v[j].y * inv * g4b[j].y,
                                                          v[j].z * inv * g4b[j].z, v[j].w * inv * g4b[j].w));
        }
    }
}
template <typename T>
void launch_resid_norm(cudaStream_t st, float* h, const float* part, int n_split, int d, const T* gain, float eps,
                       void* act, int r0, int m, unsigned int* clear16, const T* gain2, void* act2) {
    if (!gain || !act2) gain2 = nullptr;
    if (gain2) {   // draft steps only: at most 8 rows
        launch_k(k_resid_norm<T, false, true>, dim3(m), dim3(kNormThreads), 0, st, h, part, n_split, d, gain, eps, act, r0, clear16, gain2, act2);
        return;
    }
    if (r0 + m > kMaxW) launch_k(k_resid_norm<T, true, false>, dim3(m), dim3(kNormThreads), 0, st, h, part, n_split, d, gain, eps, act, r0, clear16, gain2, act2);
    else launch_k(k_resid_norm<T, false, false>, dim3(m), dim3(kNormThreads), 0, st, h, part, n_split, d, gain, eps, act, r0, clear16, gain2, act2);
}

// ------------------------------------------------------------------------------------------------
// Sum the QKV split-K partials, rotate q and k (rotate-half pairing, angle = pos * base^(-2i/hd)),
// write q (fp32) and append k, v to the paged cache in the storage dtype.
// grid = (H + 2 Hkv, m), block = hd/2 threads (one rotation pair each).
// ------------------------------------------------------------------------------------------------
struct RopeFreq { double inv_freq[64]; };
__global__ void k_rope_table(float2* tab, int n_pos, int half, RopeFreq f) {
    int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx < n_pos * half) tab[idx] = rope_cos_sin(f.inv_freq, idx / half, idx % half);
}
void launch_rope_table(cudaStream_t st, float2* tab, int n_pos, int half, const double* inv_freq) {
    RopeFreq f{};
    for (int i = 0; i < half; ++i) f.inv_freq[i] = inv_freq[i];
    k_rope_table<<<(n_pos * half + 255) / 256, 256, 0, st>>>(tab, n_pos, half, f);
}

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
    const int blk = row / kMaxW;   // partials of rows beyond the first 8 (wide prefill passes): [block][split][8][ntot]
    const float* p0 = a.qkv + ((size_t)blk * a.n_split * kMaxW + (row - blk * kMaxW)) * ntot + col + i;
    float x0 = sum_splits(p0, (size_t)kMaxW * ntot, a.n_split);
    float x1 = sum_splits(p0 + half, (size_t)kMaxW * ntot, a.n_split);
    bool is_v = head >= a.H + a.Hkv;
    if (!is_v) rope_apply(rope_fetch(a.inv_freq, a.rope_tab, half, pos, i), x0, x1);
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
// The same for the many rows of a wide prefill pass: four rotation pairs per thread (128-bit loads and stores), eight
// heads per block.  grid = (ceil((H + 2 Hkv) / 8), m), block = 8 * hd / 8 threads.  Same arithmetic, same results.
template <typename T>
__global__ void k_rope_append_wide(RopeArgs a) {
    pdl_trigger();
    pdl_wait();
    const int half = a.hd >> 1, per_head = half >> 2;            // threads per head
    const int head = blockIdx.x * 8 + threadIdx.x / per_head;
    if (head >= a.H + 2 * a.Hkv) return;
    const int i = (threadIdx.x % per_head) * 4;                  // first of this thread's four rotation pairs
    const int row = a.r0 + blockIdx.y;
    const int pos = a.pos0 + row;
    const int qd = a.H * a.hd, kvd = a.Hkv * a.hd, ntot = qd + 2 * kvd;
    const int col = head * a.hd;
    const int blk = row / kMaxW;
    const float* p0 = a.qkv + ((size_t)blk * a.n_split * kMaxW + (row - blk * kMaxW)) * ntot + col + i;
    const size_t stride4 = (size_t)kMaxW * ntot / 4;
    float4 x0 = sum_splits4(reinterpret_cast<const float4*>(p0), stride4, a.n_split);
    float4 x1 = sum_splits4(reinterpret_cast<const float4*>(p0 + half), stride4, a.n_split);
    const bool is_v = head >= a.H + a.Hkv;
    if (!is_v) {
        rope_apply(rope_fetch(a.inv_freq, a.rope_tab, half, pos, i), x0.x, x1.x);
        rope_apply(rope_fetch(a.inv_freq, a.rope_tab, half, pos, i + 1), x0.y, x1.y);
        rope_apply(rope_fetch(a.inv_freq, a.rope_tab, half, pos, i + 2), x0.z, x1.z);
        rope_apply(rope_fetch(a.inv_freq, a.rope_tab, half, pos, i + 3), x0.w, x1.w);
    }
    if (head < a.H) {
        float* q = a.q + (size_t)row * qd + col;
        *reinterpret_cast<float4*>(q + i) = x0;
        *reinterpret_cast<float4*>(q + i + half) = x1;
    } else {
        const int kvh = is_v ? head - a.H - a.Hkv : head - a.H;
        T* cache = reinterpret_cast<T*>(is_v ? a.v_cache : a.k_cache);
        const int page = a.page_table[pos >> a.page_shift];
        T* dst = cache + ((size_t)page * a.page + (pos & (a.page - 1))) * kvd + kvh * a.hd;
        if constexpr (sizeof(T) == 2) {   // four rounded values per 8-byte store
            auto pack4 = [](float4 x) {
                __nv_bfloat162 lo = __floats2bfloat162_rn(x.x, x.y), hi = __floats2bfloat162_rn(x.z, x.w);
                return make_uint2(*reinterpret_cast<uint32_t*>(&lo), *reinterpret_cast<uint32_t*>(&hi));
            };
            *reinterpret_cast<uint2*>(dst + i) = pack4(x0);
            *reinterpret_cast<uint2*>(dst + i + half) = pack4(x1);
        } else {
            *reinterpret_cast<float4*>(dst + i) = x0;
            *reinterpret_cast<float4*>(dst + i + half) = x1;
        }
    }
}
template <typename T> void launch_rope_append(cudaStream_t st, const RopeArgs& a) {
    if (a.m > kMaxW && a.hd % 8 == 0 && a.hd <= 128) {   // wide prefill pass
        dim3 grid((a.H + 2 * a.Hkv + 7) / 8, a.m);
        launch_k(k_rope_append_wide<T>, grid, dim3(a.hd), 0, st, a);
        return;
    }
    dim3 grid(a.H + 2 * a.Hkv, a.m);
    launch_k(k_rope_append<T>, grid, dim3(a.hd / 2), 0, st, a);
}

// ------------------------------------------------------------------------------------------------
// Decode attention over the paged KV cache, split over the KV length into chunks of 128 positions
// whose boundaries depend on absolute positions only (so a row's result never depends on its
// companions).  grid = (Hkv, n_chunks), 8 warps: two per 32-position block (positions base + 32 v .. + 31), each
// taking half of the (row, query head) pairs.
//   1. the block's 32 K rows (first warp) and 32 V rows (second warp) are staged in shared memory once, one TMA
//      row copy each on the block's mbarrier; they serve every query head of the KV group and every row: K and V
//      leave HBM once per layer;
//   2. q.k with one position per lane (no reduction per dot product); the softmax max and sum
//      over the 32 positions are warp-shuffle reductions;
//   3. P.V with one channel group per lane, probabilities broadcast from shared memory.
// A warp sweeps its pairs PG at a time.  Per-block partials (max, sum, out) are merged in block order into one
// partial per (chunk, row, head); the chunks are merged by k_attn_combine or, in the fused kernel, by the cluster.
// ------------------------------------------------------------------------------------------------
constexpr int kMaxPairGroup = 8;

// Shared-memory layout of k_attn_partial: rotated queries [Ppad][HD] fp32 | K tiles [4][32][padded row] | V tiles
// [4][32][row] | probabilities per warp [PG][32] | block partials [4][Ppad][HD+2].
// Where it fits, a block's partial is written over the block's own K tile once its warps are done with the scores.
struct AttnLayout {
    int Ppad, rowb_k, rowb_v;
    size_t off_k, off_v, off_p, off_mrg, total;
    bool alias;
    __host__ __device__ AttnLayout(int P, int HD, int elt, int PG, int WPB) {
        Ppad = (P + PG - 1) / PG * PG;
        rowb_k = HD * elt + 16;      // padded pitch: lane-per-row 16-byte reads of K are conflict-free
        rowb_v = HD * elt;           // V is read a whole row per warp
        off_k = (size_t)Ppad * HD * 4;
        off_v = off_k + (size_t)kPosWarps * 32 * rowb_k;
        off_p = off_v + (size_t)kPosWarps * 32 * rowb_v;
        off_mrg = off_p + (size_t)kPosWarps * WPB * PG * 32 * 4;
        // only where every warp makes at most one sweep: a second sweep would read the K tile again
        alias = (size_t)Ppad * (HD + 2) * 4 <= (size_t)32 * rowb_k && Ppad / PG <= WPB;
        total = off_mrg + (alias ? 0 : (size_t)kPosWarps * Ppad * (HD + 2) * 4);
    }
};

// mbarrier wait that lets the hardware park the thread for up to `ns` nanoseconds instead of spinning
__device__ __forceinline__ bool mbar_try_wait_parked(uint32_t bar, uint32_t parity, uint32_t ns) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"(ns)
        : "memory");
    return ok != 0;
}

// PG = (row, query head) pairs handled per sweep over a staged block: 1, 2, 4 or 8; the pair count is padded to a
// multiple of it (padding pairs compute on zero queries and are never written), so the inner loops carry no
// run-time predicates and each K element is unpacked once for up to 8 pairs.
// WPB = warps per 32-position block: 1 (the warp takes every pair; up to 8 pairs) or 2 (the groups of 8 pairs are
// split between two warps; grouped-query models with several rows).
// kFront false: the rotated queries and every cached row come from memory (launch_rope_append ran before).
// kFront true : the kernel also does what precedes it.  q is summed from the QKV split-K partials and rotated here
//          (every chunk CTA redoes it: a few hundred values); the CTA whose chunk holds the new positions sums,
//          rotates and rounds their K and V, appends them to the cache and puts them straight into its staged tile.
// The chunk partials go to global memory for k_attn_combine.  Same arithmetic in the same order in both forms and in
// the one-launch cluster kernel of the short contexts (attn_cluster.cu): bit-identical results.
template <typename T, int HD, int PG, bool kFront, int WPB>
__global__ void __launch_bounds__(kPosWarps * WPB * 32) k_attn_partial(AttnArgs a) {
    constexpr int kPairGroup = PG;
    constexpr int E = HD / 32;                       // channels per lane in P.V
    constexpr int EPP = 16 / (int)sizeof(T);         // elements per 16-byte piece
    constexpr int PPR = HD / EPP;                    // pieces per K/V row
    constexpr int ROWB_K = HD * (int)sizeof(T) + 16, ROWB_V = HD * (int)sizeof(T);
    extern __shared__ __align__(16) unsigned char smem[];
    pdl_trigger();
    const int gs = a.gsplit > 1 ? a.gsplit : 1;      // CTAs that share a KV head's query heads
    const int kvh = (int)blockIdx.x / gs, gsub = (int)blockIdx.x - kvh * gs, c = blockIdx.y;
    const int pos_pred0 = a.pos_pred0 >= 0 ? a.pos_pred0 : a.pos0 + a.r0;   // separate form: first position the preceding RoPE/append launch wrote
    if (!kFront && a.n_blocks > 1) {                 // several blocks of 8 rows in one launch: this CTA's block
        const int blk = blockIdx.z;
        a.q += (size_t)blk * kMaxW * a.H * HD;
        a.part += (size_t)blk * a.part_block_stride;
        a.pos0 += blk * kMaxW;
        if (c * kAttnChunk > a.pos0 + a.r0 + a.m - 1) return;   // a chunk beyond this block's last position
    }
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = a.H / a.Hkv / gs, P = a.m * G;     // this CTA's query heads of the group; pair p = i * G + g: row r0 + i, query head head0 + g
    const int head0 = kvh * (a.H / a.Hkv) + gsub * G;
    const GroupDiv divG(G);
    const int kvd = a.Hkv * HD, qd = a.H * HD;
    const AttnLayout lay(P, HD, (int)sizeof(T), PG, WPB);
    const int Ppad = lay.Ppad;
    float* q_s = reinterpret_cast<float*>(smem);                                   // [Ppad][HD]
    unsigned char* k_tiles = smem + lay.off_k;
    unsigned char* v_tiles = smem + lay.off_v;
    const int v = warp & (kPosWarps - 1), hsel = warp / kPosWarps;   // position block; which share of the pair groups
    unsigned char* K_w = k_tiles + (size_t)v * 32 * ROWB_K;
    unsigned char* V_w = v_tiles + (size_t)v * 32 * ROWB_V;
    float* P_w = reinterpret_cast<float*>(smem + lay.off_p) + warp * PG * 32;       // [PG][32]
    // block partial of block w: [Ppad][HD+2]
    auto mrg_blk = [&](int w) -> float* {
        return lay.alias ? reinterpret_cast<float*>(k_tiles + (size_t)w * 32 * ROWB_K)
                         : reinterpret_cast<float*>(smem + lay.off_mrg) + (size_t)w * Ppad * (HD + 2);
    };
    __shared__ __align__(8) unsigned long long stage_bar[kPosWarps];
    if (threadIdx.x < kPosWarps) mbar_init(smem_u32(&stage_bar[threadIdx.x]), WPB);   // one arrival per warp of the block
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");

    const int pos_last = a.pos0 + a.r0 + a.m - 1;
    const int pos_new0 = kFront ? a.pos0 + a.r0 : pos_last + 1;   // first position whose K,V this launch creates
    const int tbase = c * kAttnChunk + v * 32;
    const int my_t = tbase + lane;
    // The page table is set up when the context is created (or, for the stateless call, before the call)
    // and no kernel of a launch sequence writes it: like the weights it may be read before the wait.
    int my_page = 0;
    if (my_t < pos_new0) my_page = a.page_table[my_t >> a.page_shift];
    // Rows of EARLIER steps of this layer (positions below pos_done) are complete when this kernel starts: between such
    // steps the stream holds a launch without programmatic overlap (the embedding kernel that starts every step, or
    // the clear of a stateless call).  Their copies -- the long, cold loads of this kernel -- start before the
    // grid-dependency wait.  Separate form: the RoPE/append kernel right before this one wrote the rows from
    // pos_done on; they are staged after the wait, on the same barrier (the warp arrives with the second batch).
    const int pos_done = kFront ? pos_new0 : pos_pred0;
    __syncthreads();   // barriers initialised
    // 1. stage the block's K and V rows: one TMA copy per row of an earlier launch (two warps per block: the first
    //    takes K, the second V); rows beyond the last position are zeroed (their probabilities are 0, but
    //    0 * garbage must stay 0); rows this launch creates are written in step 2
    constexpr uint32_t kRowBytes = HD * (uint32_t)sizeof(T);
    const int which0 = WPB == 2 ? hsel : 0, which1 = WPB == 2 ? hsel + 1 : 2;   // 0 = K, 1 = V
    {
        const bool early = my_t < pos_done;
        const uint32_t bar = smem_u32(&stage_bar[v]);
        const unsigned n_early = __popc(__ballot_sync(0xffffffffu, early));
        if (lane == 0) {
            if (kFront) mbar_expect_tx(bar, (uint32_t)(which1 - which0) * n_early * kRowBytes);
            else mbar_expect_tx_only(bar, (uint32_t)(which1 - which0) * n_early * kRowBytes);
        }
        __syncwarp();
        for (int which = which0; which < which1; ++which) {
            unsigned char* row = which ? V_w + lane * ROWB_V : K_w + lane * ROWB_K;
            if (early) {
                const T* src = reinterpret_cast<const T*>(which ? a.v_cache : a.k_cache) +
                               ((size_t)my_page * a.page + (my_t & (a.page - 1))) * kvd + (size_t)kvh * HD;
                bulk_load(smem_u32(row), src, kRowBytes, bar);
            } else if (my_t > pos_last) {
#pragma unroll
                for (int j = 0; j < (int)kRowBytes / 16; ++j) reinterpret_cast<uint4*>(row)[j] = make_uint4(0u, 0u, 0u, 0u);
            }
        }
    }
    pdl_wait();
    if (!kFront) {   // the rows the RoPE/append kernel just wrote
        const bool late = my_t >= pos_done && my_t < pos_new0;
        const uint32_t bar = smem_u32(&stage_bar[v]);
        const unsigned n_late = __popc(__ballot_sync(0xffffffffu, late));
        if (lane == 0) mbar_expect_tx(bar, (uint32_t)(which1 - which0) * n_late * kRowBytes);
        __syncwarp();
        if (late) {
            for (int which = which0; which < which1; ++which) {
                unsigned char* row = which ? V_w + lane * ROWB_V : K_w + lane * ROWB_K;
                const T* src = reinterpret_cast<const T*>(which ? a.v_cache : a.k_cache) +
                               ((size_t)my_page * a.page + (my_t & (a.page - 1))) * kvd + (size_t)kvh * HD;
                bulk_load(smem_u32(row), src, kRowBytes, bar);
            }
        }
    }
    // 2. while those copies fly: q, and (front end) the new positions' K and V
    for (int idx = P * HD + threadIdx.x; idx < Ppad * HD; idx += blockDim.x) q_s[idx] = 0.f;   // padding pairs
    if (kFront && PG >= 4) {
        // Wide rounds: two neighbouring rotation pairs per work item (8-byte loads of the partial sums, packed stores), as in
        // the cluster kernel: every chunk CTA redoes the q rotation, and this halves its passes over the items.
        constexpr int half = HD / 2, VEC = 2, hv = half / VEC, per_pos = HD / VEC;
        const int ntot = qd + 2 * kvd;
        const size_t sstride = (size_t)kMaxW * ntot;
        const int lo = max(pos_new0, c * kAttnChunk), hi = min(pos_last, c * kAttnChunk + kAttnChunk - 1);
        const int n_q = P * hv, n_items = n_q + max(hi - lo + 1, 0) * per_pos;
        for (int idx = threadIdx.x; idx < n_items; idx += blockDim.x) {
            int kind, pos, e2, p = 0;   // kind 0: q pairs of (row, head) pair p; 1: K pairs; 2: V pairs of position pos
            if (idx < n_q) {
                p = idx / hv;
                kind = 0; pos = a.pos0 + a.r0 + divG(p); e2 = (idx - p * hv) * VEC;
            } else {
                const int j = idx - n_q, e = (j % per_pos) * VEC;
                kind = e >= half ? 2 : 1; pos = lo + j / per_pos; e2 = e >= half ? e - half : e;
            }
            const float* src = a.qkv + (size_t)(pos - a.pos0) * ntot +
                               (kind == 0 ? (head0 + (p - divG(p) * G)) * HD : qd + (kind == 2 ? kvd : 0) + kvh * HD) + e2;
            const float2 lo2 = sum_splits2(src, sstride, a.n_split), hi2 = sum_splits2(src + half, sstride, a.n_split);
            float x0[VEC] = {lo2.x, lo2.y}, x1[VEC] = {hi2.x, hi2.y};
            if (kind != 2) {
#pragma unroll
                for (int v2 = 0; v2 < VEC; ++v2) rope_apply(rope_fetch(a.inv_freq, a.rope_tab, half, pos, e2 + v2), x0[v2], x1[v2]);
            }
            if (kind == 0) {
                store_run<float, VEC>(q_s + p * HD + e2, x0);
                store_run<float, VEC>(q_s + p * HD + e2 + half, x1);
            } else {
                const bool is_v = kind == 2;
                const int page = a.page_table[pos >> a.page_shift];
                T* cache = reinterpret_cast<T*>(const_cast<void*>(is_v ? a.v_cache : a.k_cache));
                T* dst = cache + ((size_t)page * a.page + (pos & (a.page - 1))) * kvd + (size_t)kvh * HD;
                if (gsub == 0) {   // one of the CTAs that share the KV head appends; all of them put the rows in their tile
                    store_run<T, VEC>(dst + e2, x0);
                    store_run<T, VEC>(dst + e2 + half, x1);
                }
                const int tl = pos - c * kAttnChunk;
                T* srow = reinterpret_cast<T*>(is_v ? v_tiles + (size_t)tl * ROWB_V : k_tiles + (size_t)tl * ROWB_K);
                store_run<T, VEC>(srow + e2, x0);
                store_run<T, VEC>(srow + e2 + half, x1);
            }
        }
    } else if (kFront) {
        constexpr int half = HD / 2;
        constexpr int kBatch = 1;   // work items whose partial sums are requested together: one (see k_attn_cluster; here 4 were 0.7-2.7 us per layer slower)
        const int ntot = qd + 2 * kvd;
        const size_t sstride = (size_t)kMaxW * ntot;
        // work items: P * half rotation pairs of q, then, for each new position of this chunk, half rotation pairs
        // of K and half element pairs of V (rounded to the storage type, written to the cache and into the staged
        // tile of the block that owns the position)
        const int lo = max(pos_new0, c * kAttnChunk), hi = min(pos_last, c * kAttnChunk + kAttnChunk - 1);
        const int n_q = P * half, n_items = n_q + max(hi - lo + 1, 0) * HD;
        struct Item { int kind, pos, e2, p; };   // kind 0: q pair of (row, head) pair p; 1: K pair; 2: V pair of position pos
        auto item_of = [&](int idx) -> Item {
            if (idx < n_q) {
                int p = idx / half;
                return Item{0, a.pos0 + a.r0 + divG(p), idx - p * half, p};
            }
            int j = idx - n_q, it = j % HD;
            return Item{it >= half ? 2 : 1, lo + j / HD, it >= half ? it - half : it, 0};
        };
        for (int base = threadIdx.x; base < n_items; base += kBatch * blockDim.x) {
            // everything a thread's items need from memory is requested before the first value is used
            float x0[kBatch], x1[kBatch];
            float2 cs[kBatch];
            int page[kBatch];
#pragma unroll
            for (int u = 0; u < kBatch; ++u) {
                int idx = base + u * blockDim.x;
                x0[u] = x1[u] = 0.f;
                cs[u] = make_float2(1.f, 0.f);
                page[u] = 0;
                if (idx < n_items) {
                    const Item it = item_of(idx);
                    const float* p0 = a.qkv + (size_t)(it.pos - a.pos0) * ntot +
                                      (it.kind == 0 ? (head0 + (it.p - divG(it.p) * G)) * HD : qd + (it.kind == 2 ? kvd : 0) + kvh * HD) + it.e2;
                    x0[u] = sum_splits(p0, sstride, a.n_split);
                    x1[u] = sum_splits(p0 + half, sstride, a.n_split);
                    if (it.kind != 2) cs[u] = rope_fetch(a.inv_freq, a.rope_tab, half, it.pos, it.e2);
                    if (it.kind != 0) page[u] = a.page_table[it.pos >> a.page_shift];
                }
            }
#pragma unroll
            for (int u = 0; u < kBatch; ++u) {
                int idx = base + u * blockDim.x;
                if (idx >= n_items) continue;
                const Item it = item_of(idx);
                if (it.kind != 2) rope_apply(cs[u], x0[u], x1[u]);
                if (it.kind == 0) {
                    q_s[it.p * HD + it.e2] = x0[u];
                    q_s[it.p * HD + it.e2 + half] = x1[u];
                } else {
                    const bool is_v = it.kind == 2;
                    const T y0 = from_f32<T>(x0[u]), y1 = from_f32<T>(x1[u]);
                    T* cache = reinterpret_cast<T*>(const_cast<void*>(is_v ? a.v_cache : a.k_cache));
                    T* dst = cache + ((size_t)page[u] * a.page + (it.pos & (a.page - 1))) * kvd + (size_t)kvh * HD;
                    if (gsub == 0) {   // one of the CTAs that share the KV head appends; all of them put the rows in their tile
                        dst[it.e2] = y0;
                        dst[it.e2 + half] = y1;
                    }
                    int tl = it.pos - c * kAttnChunk;
                    T* srow = reinterpret_cast<T*>(is_v ? v_tiles + (size_t)tl * ROWB_V : k_tiles + (size_t)tl * ROWB_K);
                    srow[it.e2] = y0;
                    srow[it.e2 + half] = y1;
                }
            }
        }
    } else {
        for (int idx = threadIdx.x; idx < P * HD; idx += blockDim.x) {
            int p = idx / HD, e = idx - p * HD;
            int i = divG(p), g = p - i * G;
            q_s[idx] = a.q[(size_t)(a.r0 + i) * qd + (head0 + g) * HD + e];
        }
    }
    {   // bounded wait for this block's copies
        const uint32_t bar = smem_u32(&stage_bar[v]);
        if (!mbar_try_wait(bar, 0)) {
            const unsigned long long t0 = clock64();
            while (!mbar_try_wait_parked(bar, 0, 2000u)) {
                if (clock64() - t0 > kStageWaitCycles) {
                    if (a.status) atomicExch(a.status, 5u);
                    break;
                }
            }
        }
    }
    __syncthreads();   // q_s, the rows of step 2 and every block's tiles are complete

    const float scale = attn_score_scale(HD);
    // this warp's share of the pair groups
    const int n_grp = Ppad / PG, grp_split = WPB == 2 ? (n_grp + 1) / 2 : n_grp;
    const int pg_begin = hsel ? grp_split * PG : 0, pg_end = hsel ? Ppad : grp_split * PG;
    // Where the block partial goes over the K tile and two warps share the block, both must be done with the scores
    // first: a named barrier of the block's two warps, which EVERY warp executes exactly once (the layout allows that
    // overlay only if no warp makes more than one sweep; a warp without pairs arrives after the loop).
    const bool pair_barrier = WPB == 2 && lay.alias;
    bool arrived = false;
    for (int pg = pg_begin; pg < pg_end; pg += kPairGroup) {
        // ---- scores: lane = position ----
        float2 sc2[kPairGroup];   // per pair: the sums over the even and over the odd channels (attn_score_step)
#pragma unroll
        for (int pp = 0; pp < kPairGroup; ++pp) sc2[pp] = make_float2(0.f, 0.f);
#pragma unroll 2
        for (int piece = 0; piece < PPR; ++piece) {
            float kf[EPP];
            unpack16<T>(*reinterpret_cast<const uint4*>(K_w + lane * ROWB_K + piece * 16), kf);
            // the pairs' chains are independent and interleaved
#pragma unroll
            for (int v4 = 0; v4 < EPP / 4; ++v4) {
                float4 qq[kPairGroup];
#pragma unroll
                for (int pp = 0; pp < kPairGroup; ++pp)
                    qq[pp] = *reinterpret_cast<const float4*>(q_s + (size_t)(pg + pp) * HD + piece * EPP + 4 * v4);
#pragma unroll
                for (int pp = 0; pp < kPairGroup; ++pp)
                    attn_score_step(qq[pp], kf[4 * v4], kf[4 * v4 + 1], kf[4 * v4 + 2], kf[4 * v4 + 3], sc2[pp]);
            }
        }
        float sc[kPairGroup];
#pragma unroll
        for (int pp = 0; pp < kPairGroup; ++pp) sc[pp] = attn_score_finish(sc2[pp]);
        // ---- softmax pieces of this warp's 32 positions (warp-shuffle max and sum) ----
        float mx[kPairGroup], ls[kPairGroup];
#pragma unroll
        for (int pp = 0; pp < kPairGroup; ++pp) {
            int i = divG(pg + pp);
            bool on = my_t <= a.pos0 + a.r0 + i;         // causal: a row sees positions <= its own
            P_w[pp * 32 + lane] = attn_block_softmax(sc[pp], scale, on, mx[pp], ls[pp]);
        }
        __syncwarp();
        // ---- out = sum_t p_t V_t: lane = channels lane*E .. lane*E+E-1 ----
        float o[kPairGroup][E];
#pragma unroll
        for (int pp = 0; pp < kPairGroup; ++pp)
#pragma unroll
            for (int e = 0; e < E; ++e) o[pp][e] = 0.f;
#pragma unroll 2
        for (int t4 = 0; t4 < 8; ++t4) {
            float vf[4][E];
#pragma unroll
            for (int tt = 0; tt < 4; ++tt) load_channels<T, E>(V_w + (t4 * 4 + tt) * ROWB_V + lane * E * (int)sizeof(T), vf[tt]);
            // per (pair, channel) one fmaf chain over the positions in order; the chains are independent and interleaved.
            // Two neighbouring channels' chains share one packed instruction (fma.rn.f32x2: two IEEE fused
            // multiply-adds, the same roundings as two scalar ones) where a lane has an even number of channels.
            float4 p4[kPairGroup];
#pragma unroll
            for (int pp = 0; pp < kPairGroup; ++pp) p4[pp] = *reinterpret_cast<const float4*>(P_w + pp * 32 + t4 * 4);
#pragma unroll
            for (int tt = 0; tt < 4; ++tt)
#pragma unroll
                for (int pp = 0; pp < kPairGroup; ++pp) {
                    const float pt = tt == 0 ? p4[pp].x : tt == 1 ? p4[pp].y : tt == 2 ? p4[pp].z : p4[pp].w;
                    fma_channels<E>(pt, vf[tt], o[pp]);
                }
        }
        __syncwarp();   // every lane is done with its K row and with P_w
        if (pair_barrier && !arrived) {   // ... and so is the block's other warp, before the block partial goes over the K tile
            asm volatile("bar.sync %0, 64;" ::"r"(1 + v) : "memory");
            arrived = true;
        }
#pragma unroll
        for (int pp = 0; pp < kPairGroup; ++pp) {
            float* dst = mrg_blk(v) + (size_t)(pg + pp) * (HD + 2);
#pragma unroll
            for (int e = 0; e < E; ++e) dst[lane * E + e] = o[pp][e];
            if (lane == 0) {
                dst[HD] = mx[pp];
                dst[HD + 1] = ls[pp];
            }
        }
    }
    if (pair_barrier && !arrived) asm volatile("bar.sync %0, 64;" ::"r"(1 + v) : "memory");
    __syncthreads();
    // merge the four blocks in block order; thread -> (pair, two channels)
    for (int idx = threadIdx.x; idx < P * (HD / 2); idx += blockDim.x) {
        const int p = idx / (HD / 2), e = (idx - p * (HD / 2)) * 2;
        const int i = divG(p), g = p - i * G;
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < kPosWarps; ++w) M = fmaxf(M, mrg_blk(w)[(size_t)p * (HD + 2) + HD]);
        float L = 0.f, O0 = 0.f, O1 = 0.f;
        if (M > -INFINITY) {
#pragma unroll
            for (int w = 0; w < kPosWarps; ++w) {
                const float* src = mrg_blk(w) + (size_t)p * (HD + 2);
                const float mw = src[HD];
                if (mw > -INFINITY) {
                    const float f = attn_block_weight(mw, M);
                    const float2 o2 = *reinterpret_cast<const float2*>(src + e);
                    L = attn_weighted_add(L, src[HD + 1], f);
                    O0 = attn_weighted_add(O0, o2.x, f);
                    O1 = attn_weighted_add(O1, o2.y, f);
                }
            }
        }
        float* dst = a.part + (((size_t)c * kMaxW + (a.r0 + i)) * a.H + head0 + g) * (HD + 2);
        *reinterpret_cast<float2*>(dst + e) = make_float2(O0, O1);
        if (e == 0) {
            dst[HD] = M;
            dst[HD + 1] = L;
        }
    }
}

// Merge of the chunk partials of one (row, query head): grid = (H, m), 8 warps, lane = hd / 32 channels.
// Two levels, both in order: warp g folds the chunks 8g .. 8g+7 of its group one after the other (all their loads are
// issued before the first use: one L2 round trip), then the first warp folds the group partials one after the other.
// A context of up to 8 chunks is one group, which is the fold the one-launch kernel does through its cluster.
template <typename T>
__global__ void __launch_bounds__(kChunkGroup * 32) k_attn_combine(AttnArgs a) {
    __shared__ float grp[kChunkGroup][128 + 2];
    pdl_trigger();
    pdl_wait();
    const int hq = blockIdx.x, row = a.r0 + blockIdx.y, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int hd = a.hd, E = hd >> 5;                // channels per lane: 1, 2 or 4
    using A = Act<T>;
    typename A::type* act_out = reinterpret_cast<typename A::type*>(a.act_out);
    if (a.n_blocks > 1) {                            // several blocks of 8 rows in one launch: this CTA's block
        const int blk = blockIdx.z;
        a.part += (size_t)blk * a.part_block_stride;
        a.pos0 += blk * kMaxW;
        act_out += (size_t)blk * A::rows * a.H * hd;
    }
    const int n_chunks = (a.pos0 + row) / kAttnChunk + 1;   // chunks that hold positions <= this row's own
    const int n_groups = (n_chunks + kChunkGroup - 1) / kChunkGroup;
    float Mf = -INFINITY, Lf = 0.f, Of[4] = {0.f, 0.f, 0.f, 0.f};   // the first warp's running result
    for (int g0 = 0; g0 < n_groups; g0 += kChunkGroup) {
        const int g = g0 + warp;
        if (g < n_groups) {
            float mc[kChunkGroup], lc[kChunkGroup], oc[kChunkGroup][4];
#pragma unroll
            for (int u = 0; u < kChunkGroup; ++u) {
                const int c = g * kChunkGroup + u;
                const bool ok = c < n_chunks;
                const float* src = a.part + (((size_t)(ok ? c : 0) * kMaxW + row) * a.H + hq) * (hd + 2);
                mc[u] = ok ? __ldcg(src + hd) : -INFINITY;
                lc[u] = ok ? __ldcg(src + hd + 1) : 0.f;
#pragma unroll
                for (int e = 0; e < 4; ++e) oc[u][e] = (ok && e < E) ? __ldcg(src + lane * E + e) : 0.f;
            }
            float M = -INFINITY, L = 0.f, O[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int u = 0; u < kChunkGroup; ++u) {
                if (mc[u] > -INFINITY) {
                    float f0, f1;
                    attn_fold(M, L, mc[u], lc[u], f0, f1);
#pragma unroll
                    for (int e = 0; e < 4; ++e) O[e] = attn_fold_out(O[e], oc[u][e], f0, f1);
                }
            }
#pragma unroll
            for (int e = 0; e < 4; ++e)
                if (e < E) grp[warp][lane * E + e] = O[e];
            if (lane == 0) {
                grp[warp][hd] = M;
                grp[warp][hd + 1] = L;
            }
        }
        __syncthreads();
        if (warp == 0) {
            const int n_here = min(kChunkGroup, n_groups - g0);
            for (int w = 0; w < n_here; ++w) {
                const float mg = grp[w][hd];
                if (mg > -INFINITY) {
                    float f0, f1;
                    attn_fold(Mf, Lf, mg, grp[w][hd + 1], f0, f1);
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        if (e < E) Of[e] = attn_fold_out(Of[e], grp[w][lane * E + e], f0, f1);
                }
            }
        }
        __syncthreads();
    }
    if (warp == 0) {
#pragma unroll
        for (int e = 0; e < 4; ++e)
            if (e < E) A::store(act_out, row, hq * hd + lane * E + e, a.H * hd, attn_finish(Of[e], Lf));
    }
}

// Returns false if the pairs do not fit in shared memory (nothing is launched then).
template <typename T, int HD, int PG, bool kFront, int WPB>
static bool launch_attn_pg(cudaStream_t st, const AttnArgs& a, dim3 grid) {
    auto kernel = k_attn_partial<T, HD, PG, kFront, WPB>;
    const int P = a.m * (a.H / a.Hkv) / (a.gsplit > 1 ? a.gsplit : 1);
    const AttnLayout lay(P, HD, (int)sizeof(T), PG, WPB);
    const dim3 block(kPosWarps * WPB * 32);
    static bool configured[kMaxDevices];             // function attributes are per device
    const int dev = current_device();
    if (dev < 0) return false;
    if (!configured[dev]) {
        cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(200 * 1024));
        configured[dev] = true;
    }
    if (lay.total > 200 * 1024) return false;
    return launch_kc(kernel, grid, block, lay.total, st, 1, a) == cudaSuccess;
}
template <typename T, int HD, bool kFront>
static bool launch_attn_partial(cudaStream_t st, const AttnArgs& a, dim3 grid) {
    const int P = a.m * (a.H / a.Hkv) / (a.gsplit > 1 ? a.gsplit : 1);
    // Two warps per 32-position block share the pairs (latency hides behind warps, not behind instruction-level
    // parallelism: one warp per block with twice the pairs measured slower at every context length); pairs per sweep =
    // what one of the two warps gets, padded to 1, 2, 4 or 8.
    if (P > 8) return launch_attn_pg<T, HD, 8, kFront, 2>(st, a, grid);
    if (P > 4) return launch_attn_pg<T, HD, 4, kFront, 2>(st, a, grid);
    if (P > 2) return launch_attn_pg<T, HD, 2, kFront, 2>(st, a, grid);
    return launch_attn_pg<T, HD, 1, kFront, 2>(st, a, grid);   // one pair: the second warp still stages the V rows
}

template <typename T> bool launch_attention(cudaStream_t st, const AttnArgs& a) {
    const int nz = a.n_blocks > 1 ? a.n_blocks : 1;
    int n_chunks = (a.pos0 + a.r0 + (nz - 1) * kMaxW + a.m - 1) / kAttnChunk + 1;   // up to the last block's last position
    dim3 grid(a.Hkv, n_chunks, nz);
    bool ok;
    switch (a.hd) {
        case 32: ok = launch_attn_partial<T, 32, false>(st, a, grid); break;
        case 64: ok = launch_attn_partial<T, 64, false>(st, a, grid); break;
        default: ok = launch_attn_partial<T, 128, false>(st, a, grid); break;
    }
    if (!ok) return false;
    launch_attention_combine<T>(st, a);
    return true;
}

template <typename T> void launch_attention_combine(cudaStream_t st, const AttnArgs& a) {
    const int nz = a.n_blocks > 1 ? a.n_blocks : 1;
    launch_k(k_attn_combine<T>, dim3(a.H, a.m, nz), dim3(kChunkGroup * 32), 0, st, a);
}

// Contexts of any length in two launches: the chunk kernel with its front end (RoPE, cache append) and the chunk merge.
template <typename T> bool launch_attention_front(cudaStream_t st, const AttnArgs& a0) {
    if (a0.n_blocks > 1) return false;
    int n_chunks = (a0.pos0 + a0.r0 + a0.m - 1) / kAttnChunk + 1;
    // Grouped-query models: a KV head's query heads over 2 or 4 CTAs (see launch_attention_fused), for two reasons.
    // (1) Many pairs: beyond 16 (row, head) pairs a CTA needs a second sweep per warp, loses the overlay of its block
    //     partials on the K tile and with it all but one of its places on an SM (Llama-3 geometry, 6 rows: 131 us per
    //     layer against 108 at 4 rows): split until a CTA has at most 16, and on to at most 8 (three CTAs per SM instead
    //     of two) where that does not add a wave of CTAs.
    // (2) Few CTAs: split further while the grid stays within two CTAs per SM; beyond that the copies of the KV rows that
    //     every CTA of a group stages cost more than the shorter sweeps save (one row, 3000 positions: 97.4 vs 95.9 us).
    // Measured on the Llama-3 geometry, us per layer unsplit / chosen: 2500 positions 8 rows 140 / 114, 4 rows 108 / 104;
    // 8192 positions 8 rows 193 / 164, 6 rows 176 / 162.  The choice depends on the number of rows, the result does not.
    AttnArgs a = a0;
    const int Gfull = a.H / a.Hkv, sms = device_sm_count(), pairs = a.m * Gfull;
    auto waves = [&](int gs) {   // rounds of resident CTAs the grid needs with that split
        const int pc = pairs / gs, pg = pc > 8 ? 8 : pc > 4 ? 4 : pc > 2 ? 2 : 1;
        const AttnLayout lay(pc, a.hd, (int)sizeof(T), pg, 2);
        int per_sm = (int)((228 * 1024) / (lay.total + 1024));
        const int by_regs = pc > 8 ? 2 : 3;          // the 8-pair sweep needs twice the registers
        per_sm = per_sm < 1 ? 1 : per_sm > by_regs ? by_regs : per_sm;
        return (a.Hkv * gs * n_chunks + per_sm * sms - 1) / (per_sm * sms);
    };
    int gs = 1;
    while (gs < 4 && Gfull % (2 * gs) == 0 && pairs / gs > 16) gs *= 2;
    if (gs < 4 && Gfull % (2 * gs) == 0 && pairs / gs > 8 && waves(2 * gs) <= waves(gs)) gs *= 2;
    for (int g = 4; g > gs; g >>= 1)
        if (Gfull % g == 0 && a.Hkv * g * n_chunks <= 2 * sms) { gs = g; break; }
    a.gsplit = gs;
    dim3 grid(a.Hkv * a.gsplit, n_chunks);
    bool ok;
    switch (a.hd) {
        case 32: ok = launch_attn_partial<T, 32, true>(st, a, grid); break;
        case 64: ok = launch_attn_partial<T, 64, true>(st, a, grid); break;
        default: ok = launch_attn_partial<T, 128, true>(st, a, grid); break;
    }
    if (!ok) return false;
    launch_attention_combine<T>(st, a);
    return true;
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
    const float* p0 = part + (size_t)row * (2 * (size_t)F) + f;
    float g = sum_splits(p0, (size_t)kMaxW * 2 * F, n_split);
    float u = sum_splits(p0 + F, (size_t)kMaxW * 2 * F, n_split);
    float v = g / (1.f + expf(-g)) * u;
    using A = Act<T>;
    A::store(reinterpret_cast<typename A::type*>(act), row, f, F, v);
}
template <typename T> void launch_swiglu(cudaStream_t st, const float* part, int n_split, int F, void* act, int r0, int m) {
    launch_k(k_swiglu<T>, dim3((F + 255) / 256, m), dim3(256), 0, st, part, n_split, F, act, r0);
}

// ------------------------------------------------------------------------------------------------
// Greedy acceptance: the longest prefix of drafts equal to the full model's tokens, then the
// model's own token.  result = {n_emit, n_accepted_drafts, g[0..7], last emitted token}
// ------------------------------------------------------------------------------------------------
struct Drafts8 { int v[kMaxW]; };
__global__ void k_accept(const int* __restrict__ g, Drafts8 drafts, int w, int max_emit, int* __restrict__ result, Mirror mirror) {
    pdl_trigger();
    pdl_wait();
    if (threadIdx.x == 0) {
        int acc = 0;
        while (acc < w && drafts.v[acc] >= 0 && g[acc] == drafts.v[acc]) ++acc;
        int emit = acc < w ? acc + 1 : w;
        if (emit > max_emit) emit = max_emit;
        result[0] = emit;
        result[1] = acc;
        for (int i = 0; i < kMaxW; ++i) result[2 + i] = i < w ? g[i] : -1;
        result[10] = g[emit - 1];   // the token the next round starts from: the embedding kernel issued ahead reads it here
    }
    publish_results(mirror);
}
void launch_accept(cudaStream_t st, const int* g, const int* drafts8, int w, int max_emit, int* result, const Mirror& mirror) {
    Drafts8 d;
    for (int i = 0; i < kMaxW; ++i) d.v[i] = drafts8[i];
    launch_k(k_accept, dim3(1), dim3(64), 0, st, g, d, w, max_emit, result, mirror);
}

// ------------------------------------------------------------------------------------------------
// Sampling decoding (Section 4.3, decoding strategies): token = inverse CDF, in vocabulary order, of
// softmax(z / temperature), restricted to its top-p nucleus when top_p < 1, at the uniform number of the
// token's sequence position.  One cluster of 8 CTAs per row; every CTA owns a slice of whole 128-token cells.
//
//  1. slice maxima are exchanged through distributed shared memory; e_v = exp((z_v - max) / T) in fp64 goes to an
//     L2-resident scratch row (fp64 exponentials are slow on this GPU: ~35 us for 32000 of them on one SM), and,
//     for top-p, the same as a 2^40 fixed-point integer q_v.
//  2. Nucleus (top_p < 1): {v : z_v >= z*}, z* the largest logit whose upper set holds top_p of the mass (equal
//     logits enter together).  z* is found by a radix select over the order-preserving 32-bit keys of the logits,
//     11 + 11 + 10 bits from the top: each pass, every CTA histograms the integer MASS of its tokens whose key
//     matches the digits chosen so far (three 14-bit parts: 32-bit shared-memory atomics, exact and order-free),
//     then sums its share of the buckets over the 8 histograms out of its peers' shared memory and hands the sums
//     to every CTA, and every CTA scans the buckets from the top until the mass wanted is reached: the same
//     integers everywhere, so all CTAs choose the same digit.  Tokens
//     lighter than (1 - top_p) * total / V cannot decide a digit and skip the histogram.
//  3. CDF walk: every CTA sums its cells' nucleus members (a warp per cell, coalesced loads, fixed shuffle tree,
//     fp64) into the first CTA's shared memory; that CTA scans the cell sums in order, exactly one thread owns the
//     interval holding u * total (neighbouring intervals are built from the same additions), and one warp walks
//     that cell token by token.
//
// fp64 sums and exponentials: for equal logits the token can differ from an fp64 reference only by summation
// order.  Everything is a pure function of (logits, u): deterministic.  All waits are hardware barriers.
// ------------------------------------------------------------------------------------------------
constexpr int kSampleThreads = 1024;
constexpr int kSampleCell = 128;
constexpr int kSampleMaxCells = kSampleMaxVocab / kSampleCell;
constexpr int kSampleCtas = 8;
constexpr int kSelectBuckets = 2048;

__device__ __forceinline__ unsigned long long hist_mass(unsigned int h0, unsigned int h1, unsigned int h2) {
    return (unsigned long long)h0 + ((unsigned long long)h1 << 14) + ((unsigned long long)h2 << 28);
}
// larger logit <-> larger key; -0 and +0 share a key
__device__ __forceinline__ unsigned int order_key(float z) {
    const unsigned int b = __float_as_uint(z + 0.0f);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
// address of `local` (a shared-memory object of this kernel) in the CTA of cluster rank `rank`
__device__ __forceinline__ uint32_t peer_smem(const void* local, int rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_u32(local)), "r"(rank));
    return r;
}
__device__ __forceinline__ unsigned int peer_ld_u32(uint32_t addr) {
    unsigned int v;
    asm volatile("ld.shared::cluster.u32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
    return v;
}

__global__ void __launch_bounds__(kSampleThreads) k_sample(SampleArgs a) {
    pdl_trigger();
    pdl_wait();
    cluster_sync_all();   // distributed shared memory may be touched only once every CTA of the cluster has started
    // mass histogram in three 14-bit parts (a part's bucket sum stays below 2^32 for up to 262144 tokens):
    // mass of bucket b = s_hist[0][b] + (s_hist[1][b] << 14) + (s_hist[2][b] << 28)
    __shared__ unsigned int s_hist[3][kSelectBuckets];
    __shared__ double s_cell[kSampleMaxCells];          // used in the first CTA of the cluster: every cell's sum
    // during the select the same words hold the row's merged bucket masses (kSelectBuckets <= kSampleMaxCells)
    unsigned long long* s_merged = reinterpret_cast<unsigned long long*>(s_cell);
    __shared__ unsigned long long s_slice_q[kSampleCtas], s_wsum[32], s_above;
    __shared__ double s_warp[32], s_walk_run, s_walk_target;
    __shared__ float s_slice_max[kSampleCtas], s_maxw[32];
    __shared__ unsigned int s_digit;
    __shared__ int s_last, s_walk_cell;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int V = a.V, row = blockIdx.x, rank = blockIdx.y;   // cluster = (1, 8, 1): rank in the cluster = blockIdx.y
    const float* __restrict__ z = a.logits + (size_t)row * V;
    double* __restrict__ e_row = a.e + (size_t)row * V;
    unsigned long long* __restrict__ q_row = a.q + (size_t)row * V;
    const bool nucleus = a.top_p < 1.0;
    const int n_cells = (V + kSampleCell - 1) / kSampleCell;
    const int cells_per = (n_cells + kSampleCtas - 1) / kSampleCtas;
    const int c_lo = min(rank * cells_per, n_cells), c_hi = min(c_lo + cells_per, n_cells);
    const int v_lo = c_lo * kSampleCell, v_hi = min(c_hi * kSampleCell, V);

    // ---- 1. row maximum, exponentials ----
    float mx = -INFINITY;
    for (int v = v_lo + tid; v < v_hi; v += kSampleThreads) mx = fmaxf(mx, __ldcg(z + v));
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    if (lane == 0) s_maxw[warp] = mx;
    __syncthreads();
    if (tid < kSampleCtas) {                        // thread t hands this slice's maximum to the CTA of rank t
        float sm = s_maxw[0];
        for (int i = 1; i < 32; ++i) sm = fmaxf(sm, s_maxw[i]);
        asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(peer_smem(&s_slice_max[rank], tid)), "f"(sm) : "memory");
    }
    cluster_sync_all();
    mx = s_slice_max[0];
    for (int i = 1; i < kSampleCtas; ++i) mx = fmaxf(mx, s_slice_max[i]);
    unsigned long long qsum = 0ull;
    for (int v = v_lo + tid; v < v_hi; v += kSampleThreads) {
        const double ev = exp(((double)__ldcg(z + v) - (double)mx) / a.temperature);
        e_row[v] = ev;
        if (nucleus) {
            const unsigned long long qv = __double2ull_rn(ev * 1099511627776.0);   // 2^40 fixed point: integer sums are exact in any order
            q_row[v] = qv;
            qsum += qv;
        }
    }

    // ---- 2. top-p: key of the smallest logit inside the nucleus (0: every token) ----
    unsigned int kstar = 0;
    if (nucleus) {
        for (int o = 16; o > 0; o >>= 1) qsum += __shfl_xor_sync(0xffffffffu, qsum, o);
        if (lane == 0) s_wsum[warp] = qsum;
        __syncthreads();                            // also orders this CTA's e / q stores before its own loads below
        if (tid < kSampleCtas) {
            unsigned long long t = 0ull;
            for (int i = 0; i < 32; ++i) t += s_wsum[i];
            asm volatile("st.shared::cluster.u64 [%0], %1;" ::"r"(peer_smem(&s_slice_q[rank], tid)), "l"(t) : "memory");
        }
        cluster_sync_all();
        unsigned long long total_q = 0ull;
        for (int i = 0; i < kSampleCtas; ++i) total_q += s_slice_q[i];
        unsigned long long above = 0;               // mass of the keys above the current range
        unsigned long long target = (unsigned long long)ceil(a.top_p * (double)total_q);   // mass wanted
        target = target < 1ull ? 1ull : (target > total_q ? total_q : target);
        // Tokens lighter than (1 - top_p) * total / V weigh less than (1 - top_p) * total together, so the tokens at
        // or above that weight already hold the mass wanted: the lighter ones lie below the threshold logit and never
        // decide a digit (buckets above the one that mixes both kinds hold none of them).  They skip the histogram.
        const unsigned long long light = (unsigned long long)((1.0 - a.top_p) * (double)total_q / (double)V * 0.999999);
        unsigned int prefix = 0;
        int shift = 32;
        for (int pass = 0; pass < 3; ++pass) {
            const int bits = pass < 2 ? 11 : 10;
            shift -= bits;
            const unsigned int nb = 1u << bits;
            for (int i = tid; i < 3 * kSelectBuckets; i += kSampleThreads) s_hist[0][i] = 0u;
            __syncthreads();
            constexpr int kBatch = 4;   // tokens per thread per step
            for (int v0 = v_lo; v0 < v_hi; v0 += kBatch * kSampleThreads) {
                // unconditional, clamped loads first: all 2 * kBatch of them are in flight together (a load that waits
                // for the key test of its own token costs an L2 round trip per token)
                float zz[kBatch];
                unsigned long long qv[kBatch];
                unsigned int digit[kBatch];
#pragma unroll
                for (int j = 0; j < kBatch; ++j) zz[j] = __ldcg(z + min(v0 + j * kSampleThreads + tid, V - 1));
#pragma unroll
                for (int j = 0; j < kBatch; ++j) qv[j] = __ldcg(q_row + min(v0 + j * kSampleThreads + tid, V - 1));
#pragma unroll
                for (int j = 0; j < kBatch; ++j) {
                    const int v = v0 + j * kSampleThreads + tid;
                    const unsigned int k = order_key(zz[j]);
                    const bool in = v < v_hi && (pass == 0 || (k >> (shift + bits)) == prefix) && qv[j] >= light;
                    digit[j] = in ? (k >> shift) & (nb - 1) : 0xffffffffu;
                    if (!in) qv[j] = 0ull;
                }
#pragma unroll
                for (int j = 0; j < kBatch; ++j) {
                    const unsigned long long q = qv[j];
                    unsigned int p0 = (unsigned int)(q & 0x3fffull), p1 = (unsigned int)((q >> 14) & 0x3fffull),
                                 p2 = (unsigned int)(q >> 28);
                    // equal digits across the whole warp (flat or heavily tied logits) would serialise 32 atomics on
                    // one word: merge them first (exact integer reductions); otherwise one atomic per lane and part
                    const bool uniform = __all_sync(0xffffffffu, digit[j] == __shfl_sync(0xffffffffu, digit[j], 0));
                    if (uniform) {
                        p0 = __reduce_add_sync(0xffffffffu, p0);
                        p1 = __reduce_add_sync(0xffffffffu, p1);
                        p2 = __reduce_add_sync(0xffffffffu, p2);
                    }
                    if (digit[j] != 0xffffffffu && (!uniform || lane == 0)) {
                        if (p0) atomicAdd(&s_hist[0][digit[j]], p0);
                        if (p1) atomicAdd(&s_hist[1][digit[j]], p1);
                        if (p2) atomicAdd(&s_hist[2][digit[j]], p2);
                    }
                }
            }
            cluster_sync_all();                     // every CTA's histogram of this pass is complete
            {   // Bucket masses of the whole row: this CTA sums its share of the buckets (nb / 8 of them) over the 8
                // histograms and hands each sum to every CTA's table; integer sums, the same numbers everywhere.
                const int share = (int)nb / kSampleCtas;
                if (tid < share) {
                    const int b = rank * share + tid;
                    unsigned int h[kSampleCtas][3];
#pragma unroll
                    for (int r = 0; r < kSampleCtas; ++r) {
                        const uint32_t base = peer_smem(&s_hist[0][0], r);
#pragma unroll
                        for (int part = 0; part < 3; ++part) h[r][part] = peer_ld_u32(base + 4u * (uint32_t)(part * kSelectBuckets + b));
                    }
                    unsigned long long mass = 0ull;
#pragma unroll
                    for (int r = 0; r < kSampleCtas; ++r) mass += hist_mass(h[r][0], h[r][1], h[r][2]);
#pragma unroll
                    for (int r = 0; r < kSampleCtas; ++r)
                        asm volatile("st.shared::cluster.u64 [%0], %1;" ::"r"(peer_smem(&s_merged[b], r)), "l"(mass) : "memory");
                }
            }
            cluster_sync_all();                     // every CTA's table of merged bucket masses is complete
            {   // Walk the buckets from the top: a CTA-wide scan of the merged masses in descending bucket order; thread t
                // owns positions 2t and 2t+1 (position p <-> bucket nb-1-p).  Every CTA finds the same bucket.
                const int pa = 2 * tid;
                const unsigned long long m0 = pa < (int)nb ? s_merged[nb - 1 - pa] : 0ull;
                const unsigned long long m1 = pa + 1 < (int)nb ? s_merged[nb - 2 - pa] : 0ull;
                const unsigned long long mine = m0 + m1;
                unsigned long long incl = mine;
                for (int o = 1; o < 32; o <<= 1) {
                    const unsigned long long t = __shfl_up_sync(0xffffffffu, incl, o);
                    if (lane >= o) incl += t;
                }
                if (lane == 31) s_wsum[warp] = incl;
                __syncthreads();
                unsigned long long before = 0ull;
                for (int i = 0; i < warp; ++i) before += s_wsum[i];
                const unsigned long long need = target - above, excl = before + incl - mine;
                if (excl < need && need <= excl + mine) {   // the range holds at least `need`, and need >= 1
                    if (excl + m0 >= need) { s_digit = nb - 1 - pa; s_above = above + excl; }
                    else { s_digit = nb - 2 - pa; s_above = above + excl + m0; }
                }
            }
            __syncthreads();                        // s_digit, s_above; the next pass may clear this CTA's histogram:
                                                    // its peers read it before the barrier above
            above = s_above;
            prefix = (prefix << bits) | s_digit;
        }
        kstar = prefix;
        cluster_sync_all();                         // every CTA is done with its table of merged masses: the cell sums reuse it
    } else {
        __syncthreads();                            // this CTA's e stores before its own loads below
    }

    // ---- 3. cell sums of this CTA's slice, into the first CTA's table ----
    const uint32_t cell0 = peer_smem(&s_cell[0], 0);
    for (int c = c_lo + warp; c < c_hi; c += 32) {
        double s = 0.0;
#pragma unroll
        for (int j = 0; j < kSampleCell / 32; ++j) {
            const int v = c * kSampleCell + j * 32 + lane, vc = min(v, V - 1);
            const double ev = __ldcg(e_row + vc);                       // unconditional loads: in flight together
            const unsigned int kv = kstar ? order_key(__ldcg(z + vc)) : 0xffffffffu;
            if (v < V && kv >= kstar) s += ev;
        }
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        if (lane == 0)
            asm volatile("st.shared::cluster.u64 [%0], %1;" ::"r"(cell0 + 8u * (uint32_t)c), "l"(__double_as_longlong(s)) : "memory");
    }
    cluster_sync_all();                             // all cell sums are in place; every CTA's e row is visible
    if (rank != 0) return;

    // exclusive scan of the cell sums in vocabulary order: thread t owns cells [t*per, (t+1)*per)
    const int per = (n_cells + kSampleThreads - 1) / kSampleThreads;
    const int c0 = min(tid * per, n_cells), c1 = min(c0 + per, n_cells);
    double mine = 0.0;
    for (int c = c0; c < c1; ++c) mine += s_cell[c];
    double incl = mine;
    for (int o = 1; o < 32; o <<= 1) {
        double t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    double before = 0.0, total = 0.0;
    for (int i = 0; i < 32; ++i) {
        if (i < warp) before += s_warp[i];
        total += s_warp[i];
    }
    // [lower, upper] of consecutive threads tile [0, total] exactly: lower is the previous thread's upper, computed by
    // the same additions, so exactly one thread sees lower < target <= upper
    double lower = __shfl_up_sync(0xffffffffu, incl, 1);
    lower = lane == 0 ? before : before + lower;
    const double upper = before + incl;
    const double target = sample_uniform(a.seed, a.pos0 + row) * total;
    if (lower < target && target <= upper) {
        double run = lower;
        int c = c0;
        while (c < c1 - 1 && run + s_cell[c] < target) run += s_cell[c++];
        s_walk_cell = c;
        s_walk_run = run;
        s_walk_target = target;
    }
    __syncthreads();
    if (warp == 0) {
        // the cell that holds u * total, walked by one warp: lane l sums tokens 4l .. 4l+3 of the cell in order, the lane
        // sums are scanned in lane order, and the first token whose cumulative mass reaches the target is the sample
        constexpr int kPerLane = kSampleCell / 32;
        const int v0 = s_walk_cell * kSampleCell + lane * kPerLane;
        const double run0 = s_walk_run, tgt = s_walk_target;
        double ev[kPerLane];
#pragma unroll
        for (int j = 0; j < kPerLane; ++j) {
            const int v = v0 + j, vc = min(v, V - 1);
            const double e1 = __ldcg(e_row + vc);
            const unsigned int kv = kstar ? order_key(__ldcg(z + vc)) : 0xffffffffu;
            ev[j] = v < V && kv >= kstar ? e1 : 0.0;
        }
        double mine4 = 0.0;
#pragma unroll
        for (int j = 0; j < kPerLane; ++j) mine4 += ev[j];
        double incl4 = mine4;
        for (int o = 1; o < 32; o <<= 1) {
            const double t = __shfl_up_sync(0xffffffffu, incl4, o);
            if (lane >= o) incl4 += t;
        }
        double acc = run0 + (incl4 - mine4);
        int hit = -1, last_mass = -1;
#pragma unroll
        for (int j = 0; j < kPerLane; ++j) {
            if (ev[j] > 0.0) last_mass = v0 + j;
            acc += ev[j];
            if (hit < 0 && ev[j] > 0.0 && acc >= tgt) hit = v0 + j;
        }
        const unsigned int hits = __ballot_sync(0xffffffffu, hit >= 0);
        const unsigned int masses = __ballot_sync(0xffffffffu, last_mass >= 0);
        int pick;
        if (hits) pick = __shfl_sync(0xffffffffu, hit, __ffs(hits) - 1);
        else if (masses) pick = __shfl_sync(0xffffffffu, last_mass, 31 - __clz(masses));   // the walk fell an ulp short
        else pick = s_walk_cell * kSampleCell;
        if (lane == 0) {
            a.token[a.r0 + row] = pick;
            __threadfence();
        }
    }
    if (!a.mirror.host) return;                     // nothing to publish: the completion counter is not touched
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        s_last = atomicInc(a.counter, gridDim.x - 1) == gridDim.x - 1;   // one first-CTA per row; wraps back to zero
        __threadfence();
    }
    __syncthreads();
    if (s_last) publish_results(a.mirror);
}
bool launch_sample(cudaStream_t st, const SampleArgs& a) {
    return launch_kc(k_sample, dim3(a.m, kSampleCtas), dim3(kSampleThreads), 0, st, kSampleCtas, a) == cudaSuccess;
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
    template void launch_resid_norm<T>(cudaStream_t, float*, const float*, int, int, const T*, float, void*, int, int, unsigned int*, const T*, void*); \
    template void launch_rope_append<T>(cudaStream_t, const RopeArgs&);                                             \
    template bool launch_attention<T>(cudaStream_t, const AttnArgs&);                                               \
    template void launch_attention_combine<T>(cudaStream_t, const AttnArgs&);                                       \
    template bool launch_attention_front<T>(cudaStream_t, const AttnArgs&);                                         \
    template void launch_swiglu<T>(cudaStream_t, const float*, int, int, void*, int, int);
SB_INST(float)
SB_INST(__nv_bfloat16)

}  // namespace sb
