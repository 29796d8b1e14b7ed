// One-launch attention for contexts of up to 1024 cached positions (8 chunks of 128): RoPE of q and of the new K rows,
// K/V cache append, causal attention of the w <= 8 rows over the paged cache and among themselves, and the merge of the
// chunk partials through a thread-block cluster (Section 3.3: the verify pass's attention; the same kernel serves
// the draft steps and autoregressive decoding).
//
// grid = (KV heads, chunks), cluster = the chunk CTAs of a KV head, 8 warps: two per 32-position block, each taking half
// of the (row, query head) pairs.  K/V rows of earlier steps are staged by one TMA row copy each on the block's mbarrier,
// issued BEFORE the grid-dependency wait; q is summed from the QKV split-K partials and rotated here (every chunk CTA
// redoes it: a few hundred values); the CTA whose chunk holds the new positions sums, rotates and rounds their K and V,
// appends them to the cache and puts them straight into its staged tile; the chunk partials are merged, in chunk order,
// out of one another's shared memory.  The arithmetic is that of attn_common.cuh: bit-identical to the chunk kernel +
// chunk merge that longer contexts use (kernels_small.cu).  This is the latency-critical variant: at these lengths a
// CTA per SM is all there is, and every microsecond between the QKV GEMM and the output projection is on the layer's
// critical path; the layout of the long contexts' chunk kernel (3 CTAs per SM, block partials over the K tile) measured
// about 1 us per layer slower here.
#include "attn_common.cuh"

namespace sb {

constexpr int kAttnWarps = 2 * kPosWarps;     // two warps per block: each takes half of the (row, query head) pairs
constexpr int kMaxPairGroup = 8;

// PG = (row, query head) pairs handled per sweep over the staged tile: the largest of 8, 4, 2, 1 that
// divides what each warp gets, so that the inner loops carry no run-time predicates.
template <typename T, int HD, int PG>
__global__ void __launch_bounds__(kAttnWarps * 32) k_attn_cluster(AttnArgs a) {
    constexpr int kPairGroup = PG;
    constexpr int E = HD / 32;                       // channels per lane in P.V
    constexpr int EPP = 16 / (int)sizeof(T);         // elements per 16-byte piece
    constexpr int PPR = HD / EPP;                    // pieces per K/V row
    constexpr int ROWB = HD * (int)sizeof(T) + 16;   // padded row pitch: lane-per-row 16-byte reads are conflict-free
    extern __shared__ __align__(16) unsigned char smem[];
    pdl_trigger();
    const int gs = a.gsplit > 1 ? a.gsplit : 1;      // CTAs that share a KV head's query heads
    const int kvh = (int)blockIdx.x / gs, gsub = (int)blockIdx.x - kvh * gs, c = blockIdx.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = a.H / a.Hkv / gs, P = a.m * G;     // this CTA's query heads of the group; pair p = i * G + g: row r0 + i, query head head0 + g
    const int head0 = kvh * (a.H / a.Hkv) + gsub * G;
    const int kvd = a.Hkv * HD, qd = a.H * HD;
    float* q_s = reinterpret_cast<float*>(smem);                                   // [P][HD]
    unsigned char* kv_s = smem + (size_t)P * HD * 4;                                // per warp: K[32], V[32]
    const int v = warp & (kPosWarps - 1), hsel = warp / kPosWarps;   // position block; which half of the pairs
    unsigned char* K_w = kv_s + (size_t)v * 64 * ROWB;
    unsigned char* V_w = K_w + 32 * ROWB;
    float* P_w = reinterpret_cast<float*>(kv_s + (size_t)kPosWarps * 64 * ROWB) + warp * kMaxPairGroup * 32;   // [PG][32]
    float* mrg = reinterpret_cast<float*>(kv_s + (size_t)kPosWarps * 64 * ROWB) + kAttnWarps * kMaxPairGroup * 32;   // [4][P][HD+2]
    float* out_s = mrg + (size_t)kPosWarps * P * (HD + 2);   // this chunk's merged partial [P][HD+2]
    __shared__ __align__(8) unsigned long long stage_bar[kPosWarps];
    if (threadIdx.x < kPosWarps) mbar_init(smem_u32(&stage_bar[threadIdx.x]), 2);   // one arrival per warp of the block
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");

    const int pos_last = a.pos0 + a.r0 + a.m - 1;
    const int pos_new0 = a.pos0 + a.r0;   // first position whose K,V this launch creates
    const int tbase = c * kAttnChunk + v * 32;
    const int my_t = tbase + lane;
    // The page table is set up when the context is created (or, for the stateless call, before the call)
    // and no kernel of a launch sequence writes it: like the weights it may be read before the wait.
    int my_page = 0;
    if (my_t < pos_new0) my_page = a.page_table[my_t >> a.page_shift];
    // Rows of EARLIER steps of this layer (positions below pos_new0) are complete when this kernel starts: between such
    // steps the stream holds a launch without programmatic overlap (the embedding kernel that starts every step, or
    // the clear of a stateless call).  Their copies -- the long, cold loads of this kernel -- start before the
    // grid-dependency wait.
    __syncthreads();   // barriers initialised
    // 1. stage the block's K rows (first warp of the block) or V rows (second warp): one TMA copy per row of an
    //    earlier launch; rows beyond the last position are zeroed (their probabilities are 0, but 0 * garbage
    //    must stay 0); rows this launch creates are written in step 2
    constexpr uint32_t kRowBytes = HD * (uint32_t)sizeof(T);
    {
        const bool early = my_t < pos_new0;
        const uint32_t bar = smem_u32(&stage_bar[v]);
        const unsigned n_early = __popc(__ballot_sync(0xffffffffu, early));
        if (lane == 0) mbar_expect_tx(bar, n_early * kRowBytes);
        __syncwarp();
        unsigned char* row = (hsel ? V_w : K_w) + lane * ROWB;
        if (early) {
            const T* src = reinterpret_cast<const T*>(hsel ? a.v_cache : a.k_cache) +
                           ((size_t)my_page * a.page + (my_t & (a.page - 1))) * kvd + (size_t)kvh * HD;
            bulk_load(smem_u32(row), src, kRowBytes, bar);
        } else if (my_t > pos_last) {
#pragma unroll
            for (int j = 0; j < (int)kRowBytes / 16; ++j) reinterpret_cast<uint4*>(row)[j] = make_uint4(0u, 0u, 0u, 0u);
        }
    }
    // 2. while those copies fly: q, and the new positions' K and V.
    // Work items: P * half rotation pairs of q, then, for each new position of this chunk, half rotation pairs of K and
    // half element pairs of V (rounded to the storage type, written to the cache and into the staged tile of the warp
    // that owns the position).  One item's operands are requested at a time: batches of 4 (everything four items need
    // requested before the first value is used) measured 0.5-1.2 us per layer SLOWER at every width, batches of 6
    // another 1 us at one row -- the first loads leave later behind the longer address arithmetic, and that is on the
    // critical path.  For the same reason what an item needs that does not depend on the preceding kernel (its
    // addresses, its rotation angle, its page) is prepared for a thread's first item BEFORE the grid-dependency wait.
    constexpr int half = HD / 2;
    const int ntot = qd + 2 * kvd;
    const size_t sstride = (size_t)kMaxW * ntot;
    const int lo = max(pos_new0, c * kAttnChunk), hi = min(pos_last, c * kAttnChunk + kAttnChunk - 1);
    // Two forms of the same loop.  The narrow one (PG = 1: rounds of one to three rows, the latency-critical ones) is kept
    // exactly as it was measured: written as the VEC = 1 case of the wide form it compiled to code that ran 1-1.5 us per
    // layer slower, for no visible reason but its shape.
    if constexpr (PG < 2) {   // one rotation pair per work item
        const int n_q = P * half, n_items = n_q + max(hi - lo + 1, 0) * HD;
        struct Item { int kind, pos, e2, p; const float* src; float2 cs; int page; };   // kind 0: q pair of (row, head) pair p; 1: K pair; 2: V pair of position pos
        auto item_of = [&](int idx) -> Item {
            Item it;
            if (idx < n_q) {
                const int p = idx / half;
                it.kind = 0; it.pos = a.pos0 + a.r0 + p / G; it.e2 = idx - p * half; it.p = p;
            } else {
                const int j = idx - n_q, e = j % HD;
                it.kind = e >= half ? 2 : 1; it.pos = lo + j / HD; it.e2 = e >= half ? e - half : e; it.p = 0;
            }
            it.src = a.qkv + (size_t)(it.pos - a.pos0) * ntot +
                     (it.kind == 0 ? (head0 + (it.p % G)) * HD : qd + (it.kind == 2 ? kvd : 0) + kvh * HD) + it.e2;
            it.cs = it.kind != 2 ? rope_fetch(a.inv_freq, a.rope_tab, half, it.pos, it.e2) : make_float2(1.f, 0.f);
            it.page = it.kind != 0 ? a.page_table[it.pos >> a.page_shift] : 0;   // (the page table is constant: see above)
            return it;
        };
        Item first{};
        if ((int)threadIdx.x < n_items) first = item_of(threadIdx.x);
        pdl_wait();
        auto process = [&](const Item& it) {
            float x0 = sum_splits(it.src, sstride, a.n_split);
            float x1 = sum_splits(it.src + half, sstride, a.n_split);
            if (it.kind != 2) rope_apply(it.cs, x0, x1);
            if (it.kind == 0) {
                q_s[it.p * HD + it.e2] = x0;
                q_s[it.p * HD + it.e2 + half] = x1;
            } else {
                const bool is_v = it.kind == 2;
                const T y0 = from_f32<T>(x0), y1 = from_f32<T>(x1);
                T* cache = reinterpret_cast<T*>(const_cast<void*>(is_v ? a.v_cache : a.k_cache));
                T* dst = cache + ((size_t)it.page * a.page + (it.pos & (a.page - 1))) * kvd + (size_t)kvh * HD;
                if (gsub == 0) {   // one of the CTAs that share the KV head appends; all of them put the rows in their tile
                    dst[it.e2] = y0;
                    dst[it.e2 + half] = y1;
                }
                const int tl = it.pos - c * kAttnChunk;
                T* srow = reinterpret_cast<T*>(kv_s + (size_t)(tl >> 5) * 64 * ROWB + (is_v ? 32 * ROWB : 0) + (tl & 31) * ROWB);
                srow[it.e2] = y0;
                srow[it.e2 + half] = y1;
            }
        };
        // the item prepared above goes first, with its loads right behind the wait; the others, if any, through the loop
        if ((int)threadIdx.x < n_items) process(first);
        for (int idx = threadIdx.x + blockDim.x; idx < n_items; idx += blockDim.x) process(item_of(idx));
    } else {
        // Wide rounds (PG >= 2) take two neighbouring rotation pairs per item (8-byte loads of the partial sums, packed
        // stores): half as many passes over the items, and the CTA that also appends the new rows -- eight rows are 1024
        // single-pair items on 256 threads -- is what the cluster's other CTAs wait for at the merge.
        constexpr int VEC = PG >= 2 ? 2 : 1;
        constexpr int hv = half / VEC, per_pos = HD / VEC;
        const int n_q = P * hv, n_items = n_q + max(hi - lo + 1, 0) * per_pos;
        struct Item { int kind, pos, e2, p; const float* src; float2 cs[VEC]; int page; };   // kind 0: q pairs of (row, head) pair p; 1: K pairs; 2: V pairs of position pos
        auto item_of = [&](int idx) -> Item {
            Item it;
            if (idx < n_q) {
                const int p = idx / hv;
                it.kind = 0; it.pos = a.pos0 + a.r0 + p / G; it.e2 = (idx - p * hv) * VEC; it.p = p;
            } else {
                const int j = idx - n_q, e = (j % per_pos) * VEC;
                it.kind = e >= half ? 2 : 1; it.pos = lo + j / per_pos; it.e2 = e >= half ? e - half : e; it.p = 0;
            }
            it.src = a.qkv + (size_t)(it.pos - a.pos0) * ntot +
                     (it.kind == 0 ? (head0 + (it.p % G)) * HD : qd + (it.kind == 2 ? kvd : 0) + kvh * HD) + it.e2;
    #pragma unroll
            for (int v2 = 0; v2 < VEC; ++v2)
                it.cs[v2] = it.kind != 2 ? rope_fetch(a.inv_freq, a.rope_tab, half, it.pos, it.e2 + v2) : make_float2(1.f, 0.f);
            it.page = it.kind != 0 ? a.page_table[it.pos >> a.page_shift] : 0;   // (the page table is constant: see above)
            return it;
        };
        Item first{};
        if ((int)threadIdx.x < n_items) first = item_of(threadIdx.x);
        pdl_wait();
        for (int idx = threadIdx.x; idx < n_items; idx += blockDim.x) {
            const Item it = idx == (int)threadIdx.x ? first : item_of(idx);
            float x0[VEC], x1[VEC];
            if constexpr (VEC == 2) {
                const float2 lo2 = sum_splits2(it.src, sstride, a.n_split), hi2 = sum_splits2(it.src + half, sstride, a.n_split);
                x0[0] = lo2.x; x0[1] = lo2.y; x1[0] = hi2.x; x1[1] = hi2.y;
            } else {
                x0[0] = sum_splits(it.src, sstride, a.n_split);
                x1[0] = sum_splits(it.src + half, sstride, a.n_split);
            }
            if (it.kind != 2) {
    #pragma unroll
                for (int v2 = 0; v2 < VEC; ++v2) rope_apply(it.cs[v2], x0[v2], x1[v2]);
            }
            if (it.kind == 0) {
                store_run<float, VEC>(q_s + it.p * HD + it.e2, x0);
                store_run<float, VEC>(q_s + it.p * HD + it.e2 + half, x1);
            } else {
                const bool is_v = it.kind == 2;
                T* cache = reinterpret_cast<T*>(const_cast<void*>(is_v ? a.v_cache : a.k_cache));
                T* dst = cache + ((size_t)it.page * a.page + (it.pos & (a.page - 1))) * kvd + (size_t)kvh * HD;
                if (gsub == 0) {   // one of the CTAs that share the KV head appends; all of them put the rows in their tile
                    store_run<T, VEC>(dst + it.e2, x0);
                    store_run<T, VEC>(dst + it.e2 + half, x1);
                }
                const int tl = it.pos - c * kAttnChunk;
                T* srow = reinterpret_cast<T*>(kv_s + (size_t)(tl >> 5) * 64 * ROWB + (is_v ? 32 * ROWB : 0) + (tl & 31) * ROWB);
                store_run<T, VEC>(srow + it.e2, x0);
                store_run<T, VEC>(srow + it.e2 + half, x1);
            }
        }
    }
    {   // bounded wait for this block's copies
        const uint32_t bar = smem_u32(&stage_bar[v]);
        if (!mbar_try_wait(bar, 0)) {
            const unsigned long long t0 = clock64();
            while (!mbar_try_wait(bar, 0)) {
                if (clock64() - t0 > kStageWaitCycles) {
                    if (a.status) atomicExch(a.status, 5u);
                    break;
                }
            }
        }
    }
    __syncthreads();   // q_s, the rows of step 2 and both warps' tiles are complete

    const float scale = attn_score_scale(HD);
    const int P0 = (P + 1) / 2;   // pairs [0, P0) go to the first warp of a block, [P0, P) to the second
    for (int pg = hsel ? P0 : 0; pg < (hsel ? P : P0); pg += kPairGroup) {
        // ---- scores: lane = position ----
        float2 sc2[kPairGroup];   // per pair: the sums over the even and over the odd channels (attn_score_step)
#pragma unroll
        for (int pp = 0; pp < kPairGroup; ++pp) sc2[pp] = make_float2(0.f, 0.f);
#pragma unroll 2
        for (int piece = 0; piece < PPR; ++piece) {
            float kf[EPP];
            unpack16<T>(*reinterpret_cast<const uint4*>(K_w + lane * ROWB + piece * 16), kf);
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
            int i = (pg + pp) / G;
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
            for (int tt = 0; tt < 4; ++tt) {
                load_channels<T, E>(V_w + (t4 * 4 + tt) * ROWB + lane * E * (int)sizeof(T), vf[tt]);
            }
            // per (pair, channel) one fmaf chain over the positions in order, two neighbouring channels per packed instruction
#pragma unroll
            for (int pp = 0; pp < kPairGroup; ++pp) {
                const float4 p4 = *reinterpret_cast<const float4*>(P_w + pp * 32 + t4 * 4);
                fma_channels<E>(p4.x, vf[0], o[pp]);
                fma_channels<E>(p4.y, vf[1], o[pp]);
                fma_channels<E>(p4.z, vf[2], o[pp]);
                fma_channels<E>(p4.w, vf[3], o[pp]);
            }
        }
        __syncwarp();
#pragma unroll
        for (int pp = 0; pp < kPairGroup; ++pp) {
            float* dst = mrg + ((size_t)v * P + pg + pp) * (HD + 2);
#pragma unroll
            for (int e = 0; e < E; ++e) dst[lane * E + e] = o[pp][e];
            if (lane == 0) {
                dst[HD] = mx[pp];
                dst[HD + 1] = ls[pp];
            }
        }
    }
    __syncthreads();
    // merge the four warps in warp order; thread -> (pair, channel)
    for (int idx = threadIdx.x; idx < P * HD; idx += blockDim.x) {
        int p = idx / HD, e = idx - p * HD;
        int i = p / G, g = p - i * G;
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < kPosWarps; ++w) M = fmaxf(M, mrg[((size_t)w * P + p) * (HD + 2) + HD]);
        float L = 0.f, O = 0.f;
        if (M > -INFINITY) {
#pragma unroll
            for (int w = 0; w < kPosWarps; ++w) {
                const float* src = mrg + ((size_t)w * P + p) * (HD + 2);
                float mw = src[HD];
                if (mw > -INFINITY) {
                    const float f = attn_block_weight(mw, M);
                    L = attn_weighted_add(L, src[HD + 1], f);
                    O = attn_weighted_add(O, src[e], f);
                }
            }
        }
        float* dst = out_s + (size_t)p * (HD + 2);
        dst[e] = O;
        if (e == 0) {
            dst[HD] = M;
            dst[HD + 1] = L;
        }
    }
    // ---- chunk merge across the cluster (one CTA per chunk of this KV head) ----
    __syncthreads();
    cluster_sync_all();   // every chunk's partial is in its CTA's out_s
    {   // every CTA of the cluster merges its share of the (pair, channel) outputs
        const uint32_t out_local = (uint32_t)__cvta_generic_to_shared(out_s);
        constexpr int kBatch = 8;
        for (int idx = c * blockDim.x + threadIdx.x; idx < P * HD; idx += gridDim.y * blockDim.x) {
            int p = idx / HD, e = idx - p * HD;
            int i = p / G, g = p - i * G;
            int row = a.r0 + i;
            int n_chunks = (a.pos0 + row) / kAttnChunk + 1;   // chunks that hold positions <= this row's own (<= cluster size)
            float M = -INFINITY, L = 0.f, O = 0.f;
            float mc[kBatch], lc[kBatch], oc[kBatch];
#pragma unroll
            for (int u = 0; u < kBatch; ++u) {
                mc[u] = -INFINITY; lc[u] = 0.f; oc[u] = 0.f;
                if (u < n_chunks) {
                    uint32_t base;
                    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(base) : "r"(out_local + (uint32_t)(p * (HD + 2)) * 4u), "r"(u));
                    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(mc[u]) : "r"(base + (uint32_t)HD * 4u) : "memory");
                    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(lc[u]) : "r"(base + (uint32_t)(HD + 1) * 4u) : "memory");
                    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(oc[u]) : "r"(base + (uint32_t)e * 4u) : "memory");
                }
            }
#pragma unroll
            for (int u = 0; u < kBatch; ++u) {
                if (mc[u] > -INFINITY) {
                    float f0, f1;
                    attn_fold(M, L, mc[u], lc[u], f0, f1);
                    O = attn_fold_out(O, oc[u], f0, f1);
                }
            }
            using A = Act<T>;
            A::store(reinterpret_cast<typename A::type*>(a.act_out), row, (head0 + g) * HD + e, a.H * HD, attn_finish(O, L));
        }
    }
    __syncthreads();
    cluster_sync_all();   // a CTA's shared memory stays alive until its peers have read it
}

static size_t cluster_attn_smem(int P, int HD, size_t elt) {
    const int rowb = HD * (int)elt + 16;
    return (size_t)P * HD * 4 + (size_t)kPosWarps * 64 * rowb + (size_t)kAttnWarps * kMaxPairGroup * 32 * 4 +
           (size_t)kPosWarps * P * (HD + 2) * 4 + (size_t)P * (HD + 2) * 4;
}
// Returns false if the device cannot co-schedule such a cluster or the pairs do not fit (nothing is launched then).
template <typename T, int HD, int PG>
static bool launch_cluster_pg(cudaStream_t st, const AttnArgs& a, dim3 grid, size_t smem, int cluster_y) {
    auto kernel = k_attn_cluster<T, HD, PG>;
    static bool configured[kMaxDevices];             // function attributes are per device
    const int dev = current_device();
    if (dev < 0 || smem > 200 * 1024) return false;
    if (!configured[dev]) {
        cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(200 * 1024));
        configured[dev] = true;
    }
    if (cluster_y > 1) {
        static int resident_dev[kMaxDevices][9];         // per device and cluster size: clusters resident at once + 1 (0 = not asked yet)
        int* resident = resident_dev[dev];
        if (resident[cluster_y] == 0) {
            cudaLaunchConfig_t cfg{};
            cfg.gridDim = grid; cfg.blockDim = dim3(kAttnWarps * 32); cfg.dynamicSmemBytes = 200 * 1024;
            cudaLaunchAttribute at[1];
            at[0].id = cudaLaunchAttributeClusterDimension;
            at[0].val.clusterDim.x = 1; at[0].val.clusterDim.y = (unsigned)cluster_y; at[0].val.clusterDim.z = 1;
            cfg.attrs = at; cfg.numAttrs = 1;
            int n = 0;
            if (cudaOccupancyMaxActiveClusters(&n, kernel, &cfg) != cudaSuccess) { (void)cudaGetLastError(); n = 0; }
            resident[cluster_y] = n + 1;
            if (getenv("SB_DEBUG")) fprintf(stderr, "[specbound] attention clusters of %d CTAs: %d resident at once\n", cluster_y, n);
        }
        if (resident[cluster_y] - 1 < 1) return false;
    }
    return launch_kc(kernel, grid, dim3(kAttnWarps * 32), smem, st, cluster_y, a) == cudaSuccess;
}
template <typename T, int HD>
static bool launch_cluster_hd(cudaStream_t st, const AttnArgs& a, dim3 grid, int cluster_y) {
    const int P = a.m * (a.H / a.Hkv) / (a.gsplit > 1 ? a.gsplit : 1);
    size_t smem = cluster_attn_smem(P, HD, sizeof(T));
    // pairs per sweep: the largest of 8, 4, 2, 1 that divides what each of a block's two warps gets
    const int P0 = (P + 1) / 2, P1 = P - P0;
    auto divides = [&](int g) { return P0 % g == 0 && P1 % g == 0; };
    if (divides(8)) return launch_cluster_pg<T, HD, 8>(st, a, grid, smem, cluster_y);
    if (divides(4)) return launch_cluster_pg<T, HD, 4>(st, a, grid, smem, cluster_y);
    if (divides(2)) return launch_cluster_pg<T, HD, 2>(st, a, grid, smem, cluster_y);
    return launch_cluster_pg<T, HD, 1>(st, a, grid, smem, cluster_y);
}

template <typename T> bool launch_attention_fused(cudaStream_t st, const AttnArgs& a) {
    int n_chunks = (a.pos0 + a.r0 + a.m - 1) / kAttnChunk + 1;
    // up to 8 chunks: the portable cluster size.  (Clusters of 9-16 chunk CTAs, which fit the device at once only for
    // models with few KV heads, were built and measured: slower than the chunk kernel with its query-head split, e.g.
    // Llama-3 geometry at 1030 positions, 8 rows: 116.6 vs 104.8 us per layer.)
    if (n_chunks > 8) return false;
    // Grouped-query models: with few KV heads there are fewer CTAs than SMs, each doing the CUDA-core work of all its
    // group's (row, head) pairs; spread a group's query heads over 2 or 4 CTAs (every one of them stages the KV head's rows:
    // a few MB more out of L2) while the grid stays about within one CTA per SM, or within two where a CTA would
    // otherwise sweep 16 pairs or more (two CTAs of up to 8 pairs fit an SM).  Llama-3 geometry, 512 positions, us per
    // layer at 1 / 2 / 4 / 6 / 8 rows: unsplit 93.3 / 97.5 / 101.8 / 110.6 / 116.3, two CTAs per KV head 89.8 / 92.1 / 97.2 /
    // 105.2 / 103.1, four 88.9 / 89.9 / 93.0 / 98.6 / 99.1; at 900 positions four CTAs lose to two at 1-2 rows (92.1 vs
    // 89.6).  A split that cannot be launched falls back to the next smaller one.
    const int Gfull = a.H / a.Hkv, sms = device_sm_count(), pairs = a.m * Gfull;
    for (int gs = 4; gs >= 1; gs >>= 1) {
        const int ctas = a.Hkv * gs * n_chunks;
        if (Gfull % gs) continue;
        if (gs > 1 && !(ctas <= sms + sms / 8 || (pairs >= 16 && ctas <= 2 * sms))) continue;
        AttnArgs b = a;
        b.gsplit = gs;
        dim3 grid(a.Hkv * gs, n_chunks);
        bool ok;
        switch (a.hd) {
            case 32: ok = launch_cluster_hd<T, 32>(st, b, grid, n_chunks); break;
            case 64: ok = launch_cluster_hd<T, 64>(st, b, grid, n_chunks); break;
            default: ok = launch_cluster_hd<T, 128>(st, b, grid, n_chunks); break;
        }
        if (ok) return true;
    }
    return false;
}

template bool launch_attention_fused<float>(cudaStream_t, const AttnArgs&);
template bool launch_attention_fused<__nv_bfloat16>(cudaStream_t, const AttnArgs&);

}  // namespace sb
