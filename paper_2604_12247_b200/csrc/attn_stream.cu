// Decode attention over long contexts (more than 8 chunks of 128 cached positions): the chunk partials of the
// verify pass (Section 3.3: w <= 8 rows attend over the paged KV cache and among themselves).
//
// Every WARP is an independent streaming pipeline.  A work item is (KV head, 128-position chunk, slice of up to 8
// (row, query head) pairs); the warp walks its items one after the other and, inside an item, eight staging tiles of
// 32 cached rows each: the chunk's four K blocks, then its four V blocks.  Tiles go through a private ring of three
// slots filled by one TMA row copy per lane on the slot's own mbarrier, two tiles ahead of the one being consumed, so
// the copies of a warp overlap its arithmetic and the ring simply runs on into the next item; no warp ever waits for
// another one (no CTA-wide barrier in the loop).  K tiles: one position per lane, the scores of all pairs of the slice
// from one pass over the lane's row (each K element is unpacked once for up to 8 pairs), block softmax by warp
// butterflies, probabilities parked in shared memory.  After the fourth K tile the chunk maximum is known, so each V
// tile's block result (one channel group per lane) is weighted and added to the chunk partial in registers as soon as
// it is complete.  The chunk partial (max, sum, out) goes to global memory for the merge kernel.
//
// The arithmetic and its order are those of attn_common.cuh: bit-identical to the separate chunk kernel.
#include "attn_common.cuh"

namespace sb {

constexpr int kStreamSlots = 3;       // staging tiles per warp
constexpr int kStreamMaxWarps = 8;
constexpr int kStreamSmemBudget = 220 * 1024;

template <typename T, int HD, int PG> struct StreamLayout {
    static constexpr int ROWB = HD * (int)sizeof(T) + 16;          // padded row pitch: lane-per-row 16-byte reads are conflict-free
    static constexpr int kSlotBytes = 32 * ROWB;
    static constexpr int kQBytes = PG * HD * 4;                    // the slice's rotated queries [pair][HD]
    static constexpr int kPBytes = PG * kAttnChunk * 4;            // probabilities [pair][position in chunk]
    static constexpr int kMlBytes = kPosWarps * PG * 2 * 4;        // block (max, sum) [block][pair]
    static constexpr int kWarpBytes = kStreamSlots * kSlotBytes + kQBytes + kPBytes + kMlBytes;
    static_assert(kWarpBytes % 16 == 0, "per-warp region must keep 16-byte alignment");
};

__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

template <typename T, int HD, int PG>
__global__ void __launch_bounds__(kStreamMaxWarps * 32, 1) k_attn_stream(AttnArgs a, int warps_per_cta, int n_slices, int n_items) {
    using Lay = StreamLayout<T, HD, PG>;
    constexpr int E = HD / 32;                       // channels per lane in P.V
    constexpr int EPP = 16 / (int)sizeof(T);         // elements per 16-byte piece
    constexpr int PPR = HD / EPP;                    // pieces per K/V row
    constexpr int ROWB = Lay::ROWB;
    constexpr uint32_t kRowBytes = HD * (uint32_t)sizeof(T);
    extern __shared__ __align__(16) unsigned char smem[];
    __shared__ __align__(8) unsigned long long bars[kStreamMaxWarps][kStreamSlots];
    pdl_trigger();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    unsigned char* const slots = smem + (size_t)warp * Lay::kWarpBytes;
    float* const q_s = reinterpret_cast<float*>(slots + kStreamSlots * Lay::kSlotBytes);
    float* const P_s = q_s + PG * HD;
    float* const ml_s = P_s + PG * kAttnChunk;
    if (lane == 0) {
#pragma unroll
        for (int s = 0; s < kStreamSlots; ++s) mbar_init(smem_u32(&bars[warp][s]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();

    const int G = a.H / a.Hkv, P = a.m * G;          // pair p = i * G + g: row r0 + i, query head kvh * G + g
    const int kvd = a.Hkv * HD, qd = a.H * HD;
    const int pos_last = a.pos0 + a.r0 + a.m - 1;    // every position up to here is in the cache when the copies run
    const int pos_pred0 = a.pos_pred0 >= 0 ? a.pos_pred0 : a.pos0 + a.r0;   // first row the preceding launch wrote
    // items of this warp: wid, wid + total warps, ...; consecutive items sit on different SMs
    const int total_warps = (int)gridDim.x * warps_per_cta;
    const int wid = warp * (int)gridDim.x + (int)blockIdx.x;
    const int n_my = warp < warps_per_cta && wid < n_items ? (n_items - wid + total_warps - 1) / total_warps : 0;
    const int n_tiles = 8 * n_my;
    bool waited = false;                             // grid-dependency wait done
    bool gave_up = false;

    // tile n of this warp: item wid + (n / 8) * total_warps; tile 0-3 = K blocks, 4-7 = V blocks of the item's chunk
    auto item_of = [&](int k, int& kvh, int& c, int& slice) {
        const int item = wid + k * total_warps;
        slice = item % n_slices;
        const int t = item / n_slices;
        kvh = t % a.Hkv;
        c = t / a.Hkv;
    };
    // rows of a tile that an earlier step wrote may be fetched before the grid-dependency wait (see k_attn_partial)
    auto tile_is_early = [&](int n) {
        int kvh, c, slice;
        item_of(n >> 3, kvh, c, slice);
        const int last = min(c * kAttnChunk + (n & 3) * 32 + 31, pos_last);
        return last < pos_pred0;
    };
    auto issue = [&](int n) {
        int kvh, c, slice;
        item_of(n >> 3, kvh, c, slice);
        const int j = n & 3, is_v = (n >> 2) & 1;
        const int t = c * kAttnChunk + j * 32 + lane;
        const int slot = n % kStreamSlots;
        const uint32_t bar = smem_u32(&bars[warp][slot]);
        unsigned char* row = slots + (size_t)slot * Lay::kSlotBytes + lane * ROWB;
        const bool valid = t <= pos_last;
        const unsigned n_valid = __popc(__ballot_sync(0xffffffffu, valid));
        if (lane == 0) mbar_expect_tx(bar, n_valid * kRowBytes);
        __syncwarp();
        if (valid) {
            const int page = a.page_table[t >> a.page_shift];
            const T* src = reinterpret_cast<const T*>(is_v ? a.v_cache : a.k_cache) +
                           ((size_t)page * a.page + (t & (a.page - 1))) * kvd + (size_t)kvh * HD;
            bulk_load(smem_u32(row), src, kRowBytes, bar);
        } else {   // beyond the last position: probabilities are 0 there, but 0 * garbage must stay 0
#pragma unroll
            for (int b = 0; b < (int)kRowBytes / 16; ++b) reinterpret_cast<uint4*>(row)[b] = make_uint4(0u, 0u, 0u, 0u);
        }
    };

    // prologue: tiles that hold rows of earlier steps only start before the grid-dependency wait
    int next_issue = 0;
    while (next_issue < n_tiles && next_issue < kStreamSlots && tile_is_early(next_issue)) issue(next_issue++);
    pdl_wait();
    waited = true;
    (void)waited;

    const float scale = attn_score_scale(HD);
    float M[PG], L[PG], O[PG][E];
    int kvh = 0, c = 0, slice = 0;
    for (int n = 0; n < n_tiles && !gave_up; ++n) {
        const int j = n & 3, tau = n & 7;
        // the slot of tile n - 1 is free now: every lane is done with it
        __syncwarp();
        fence_proxy_async_smem();
        while (next_issue < n_tiles && next_issue < n + kStreamSlots) issue(next_issue++);
        if (tau == 0) {   // a new item: its queries (the previous item's score phase is over)
            item_of(n >> 3, kvh, c, slice);
            for (int idx = lane; idx < PG * HD / 4; idx += 32) {
                const int pp = idx / (HD / 4), e4 = idx - pp * (HD / 4);
                const int p = slice * PG + pp;
                float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
                if (p < P) {
                    const int i = p / G, g = p - i * G;
                    v = __ldcg(reinterpret_cast<const float4*>(a.q + (size_t)(a.r0 + i) * qd + (kvh * G + g) * HD) + e4);
                }
                reinterpret_cast<float4*>(q_s)[idx] = v;
            }
            __syncwarp();
        }
        {   // bounded wait for the tile's copies
            const uint32_t bar = smem_u32(&bars[warp][n % kStreamSlots]);
            const uint32_t parity = (uint32_t)(n / kStreamSlots) & 1u;
            if (!mbar_try_wait(bar, parity)) {
                const unsigned long long t0 = clock64();
                while (!mbar_try_wait(bar, parity)) {
                    if (clock64() - t0 > kStageWaitCycles) {
                        if (a.status) atomicExch(a.status, 5u);
                        gave_up = true;
                        break;
                    }
                }
            }
            gave_up = __any_sync(0xffffffffu, gave_up);
            if (gave_up) break;
        }
        __syncwarp();   // the zero rows other lanes wrote
        const unsigned char* tile = slots + (size_t)(n % kStreamSlots) * Lay::kSlotBytes;
        if (tau < 4) {
            // ---- scores of block j: lane = position ----
            const int my_t = c * kAttnChunk + j * 32 + lane;
            float sc[PG];
#pragma unroll
            for (int pp = 0; pp < PG; ++pp) sc[pp] = 0.f;
#pragma unroll 2
            for (int piece = 0; piece < PPR; ++piece) {
                float kf[EPP];
                unpack16<T>(*reinterpret_cast<const uint4*>(tile + lane * ROWB + piece * 16), kf);
#pragma unroll
                for (int pp = 0; pp < PG; ++pp) {
                    const float4* qv = reinterpret_cast<const float4*>(q_s + pp * HD + piece * EPP);
#pragma unroll
                    for (int v4 = 0; v4 < EPP / 4; ++v4) {
                        const float4 qq = qv[v4];
                        sc[pp] = fmaf(qq.x, kf[4 * v4], sc[pp]);
                        sc[pp] = fmaf(qq.y, kf[4 * v4 + 1], sc[pp]);
                        sc[pp] = fmaf(qq.z, kf[4 * v4 + 2], sc[pp]);
                        sc[pp] = fmaf(qq.w, kf[4 * v4 + 3], sc[pp]);
                    }
                }
            }
#pragma unroll
            for (int pp = 0; pp < PG; ++pp) {
                const int i = (slice * PG + pp) / G;
                const bool on = my_t <= a.pos0 + a.r0 + i;      // causal: a row sees positions <= its own
                float m, l;
                P_s[pp * kAttnChunk + j * 32 + lane] = attn_block_softmax(sc[pp], scale, on, m, l);
                if (lane == 0) {
                    ml_s[(j * PG + pp) * 2] = m;
                    ml_s[(j * PG + pp) * 2 + 1] = l;
                }
            }
            if (tau == 3) {   // all four blocks' maxima are known: the chunk's maximum and sum
                __syncwarp();
#pragma unroll
                for (int pp = 0; pp < PG; ++pp) {
                    float mx = -INFINITY;
#pragma unroll
                    for (int b = 0; b < kPosWarps; ++b) mx = fmaxf(mx, ml_s[(b * PG + pp) * 2]);
                    float ls = 0.f;
                    if (mx > -INFINITY) {
#pragma unroll
                        for (int b = 0; b < kPosWarps; ++b) {
                            const float mb = ml_s[(b * PG + pp) * 2];
                            if (mb > -INFINITY) ls = attn_weighted_add(ls, ml_s[(b * PG + pp) * 2 + 1], attn_block_weight(mb, mx));
                        }
                    }
                    M[pp] = mx;
                    L[pp] = ls;
#pragma unroll
                    for (int e = 0; e < E; ++e) O[pp][e] = 0.f;
                }
            }
        } else {
            // ---- out of block j = sum_t p_t V_t: lane = channels lane*E .. lane*E+E-1 ----
            float o[PG][E];
#pragma unroll
            for (int pp = 0; pp < PG; ++pp)
#pragma unroll
                for (int e = 0; e < E; ++e) o[pp][e] = 0.f;
#pragma unroll 2
            for (int t4 = 0; t4 < 8; ++t4) {
                float vf[4][E];
#pragma unroll
                for (int tt = 0; tt < 4; ++tt) load_channels<T, E>(tile + (t4 * 4 + tt) * ROWB + lane * E * (int)sizeof(T), vf[tt]);
#pragma unroll
                for (int pp = 0; pp < PG; ++pp) {
                    const float4 p4 = *reinterpret_cast<const float4*>(P_s + pp * kAttnChunk + j * 32 + t4 * 4);
#pragma unroll
                    for (int e = 0; e < E; ++e) {
                        o[pp][e] = fmaf(p4.x, vf[0][e], o[pp][e]);
                        o[pp][e] = fmaf(p4.y, vf[1][e], o[pp][e]);
                        o[pp][e] = fmaf(p4.z, vf[2][e], o[pp][e]);
                        o[pp][e] = fmaf(p4.w, vf[3][e], o[pp][e]);
                    }
                }
            }
#pragma unroll
            for (int pp = 0; pp < PG; ++pp) {
                const float mb = ml_s[(j * PG + pp) * 2];
                if (M[pp] > -INFINITY && mb > -INFINITY) {
                    const float f = attn_block_weight(mb, M[pp]);
#pragma unroll
                    for (int e = 0; e < E; ++e) O[pp][e] = attn_weighted_add(O[pp][e], o[pp][e], f);
                }
            }
            if (tau == 7) {   // the chunk partial of every pair of the slice
#pragma unroll
                for (int pp = 0; pp < PG; ++pp) {
                    const int p = slice * PG + pp;
                    if (p < P) {
                        const int i = p / G, g = p - i * G;
                        float* dst = a.part + (((size_t)c * kMaxW + (a.r0 + i)) * a.H + kvh * G + g) * (HD + 2);
#pragma unroll
                        for (int e = 0; e < E; ++e) dst[lane * E + e] = O[pp][e];
                        if (lane == 0) {
                            dst[HD] = M[pp];
                            dst[HD + 1] = L[pp];
                        }
                    }
                }
            }
        }
    }
    if (gave_up) {   // copies may still be in flight into this CTA's shared memory: give them time to land
        const unsigned long long t0 = clock64();
        while (clock64() - t0 < 4000000ull) {}
    }
}

template <typename T, int HD, int PG>
static bool launch_stream_pg(cudaStream_t st, const AttnArgs& a, int n_slices, int n_items) {
    using Lay = StreamLayout<T, HD, PG>;
    auto kernel = k_attn_stream<T, HD, PG>;
    int W = kStreamSmemBudget / Lay::kWarpBytes;
    if (W > kStreamMaxWarps) W = kStreamMaxWarps;
    if (W < 1) return false;
    static bool configured[kMaxDevices];
    const int dev = current_device();
    if (dev < 0) return false;
    if (!configured[dev]) {
        cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kStreamSmemBudget);
        configured[dev] = true;
    }
    const int sms = device_sm_count();
    const int grid = n_items < sms ? n_items : sms;
    return launch_kc(kernel, dim3(grid), dim3(W * 32), (size_t)W * Lay::kWarpBytes, st, 1, a, W, n_slices, n_items) == cudaSuccess;
}

template <typename T, int HD>
static bool launch_stream_hd(cudaStream_t st, const AttnArgs& a) {
    const int P = a.m * (a.H / a.Hkv);
    const int n_chunks = (a.pos0 + a.r0 + a.m - 1) / kAttnChunk + 1;
    // pairs per sweep: the smallest of 1, 2, 4, 8 that holds all pairs of a KV head, else slices of 8 (a slice's unused
    // pair slots compute on zero queries and are never written)
    const int PG = P >= 8 ? 8 : (P > 4 ? 8 : (P > 2 ? 4 : P));
    const int n_slices = (P + PG - 1) / PG;
    const int n_items = n_chunks * a.Hkv * n_slices;
    switch (PG) {
        case 1: return launch_stream_pg<T, HD, 1>(st, a, n_slices, n_items);
        case 2: return launch_stream_pg<T, HD, 2>(st, a, n_slices, n_items);
        case 4: return launch_stream_pg<T, HD, 4>(st, a, n_slices, n_items);
        default: return launch_stream_pg<T, HD, 8>(st, a, n_slices, n_items);
    }
}

template <typename T> bool launch_attention_stream(cudaStream_t st, const AttnArgs& a) {
    if (a.n_blocks > 1) return false;
    bool ok;
    switch (a.hd) {
        case 32: ok = launch_stream_hd<T, 32>(st, a); break;
        case 64: ok = launch_stream_hd<T, 64>(st, a); break;
        default: ok = launch_stream_hd<T, 128>(st, a); break;
    }
    if (!ok) return false;
    launch_attention_combine<T>(st, a);
    return true;
}

template bool launch_attention_stream<float>(cudaStream_t, const AttnArgs&);
template bool launch_attention_stream<__nv_bfloat16>(cudaStream_t, const AttnArgs&);

}  // namespace sb
