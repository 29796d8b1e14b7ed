// TMA + tcgen05 weight-streaming kernels for bf16 models (sm_100a).
//
//   out[row][n] = sum_k act[row][k] * W[n][k]        rows <= 8, W streamed from HBM exactly once
//
// The weight tile is the MMA's M operand (128 weight rows x 64 k per pipeline stage, staged by
// TMA with the 128-byte swizzle); the activations are the N operand: 16 columns = the high and
// the low bf16 halves of the 8 fp32 activation rows, so one kind::f16 MMA (M=128, N=16, K=16)
// yields W.hi and W.lo side by side in TMEM and their sum is as accurate as an fp32 product.
//
// One persistent CTA per SM: warps 0-3 = TMA producers (one issuing thread moves only ~20 B/clk
// through TMA -- a 128-byte row every ~6.5 clocks -- so four of them take every fourth pipeline
// fill to reach the HBM rate), warp 4 = MMA issuer (owns TMEM), warps 5-8 = epilogue (tcgen05.ld,
// then either split-K partial stores or, for the LM head, the online temperature-scaled softmax
// max/argmax of Eq. 2).  Work items are (row slab, k split) pairs
// chosen on the host so that every CTA streams the same number of bytes whatever the number of
// rows: the result of a row never depends on its companions.  Every wait is bounded: on expiry
// the kernel raises a status word, drains and returns.
#include <cuda.h>

#include <cstdio>
#include <cstring>

#include "gemm_tc.cuh"

namespace sb {

constexpr int kMaxStages = 12;                // pipeline depth is a launch parameter (tuned per use)
constexpr int kBK = 64;                       // k elements per stage (128 bytes: one swizzle row)
constexpr int kTileRows = 128;                // MMA M
constexpr int kStageA = kTileRows * kBK * 2;  // 16 KB
constexpr int kStageB = 16 * kBK * 2;         // 2 KB
constexpr int kProducers = 4;                 // producer warps
constexpr int kTcThreads = (kProducers + 5) * 32;
static int smem_bytes(int stages, int nb = 1) { return stages * (kStageA + nb * kStageB) + 1024 /*alignment slack*/ + 256 /*barriers*/; }
// Wide mode (prefill): kWideBlocks blocks of 8 activation rows ride through one launch (MMA N = 16 per block); a stage
// is 16 KB of weights + 2 KB per block of activations, so one CTA per SM with 4 stages (>= the number of producers).
constexpr int kWideStages = 4;
static_assert(kWideStages * (kStageA + kWideBlocks * kStageB) + 1280 <= 227 * 1024, "wide stages exceed shared memory");
static_assert(2 * 16 * kWideBlocks <= 512, "two wide accumulators exceed tensor memory");
// Two CTAs per SM (each with its own producers, MMA issuer and TMEM accumulators) stream measurably
// faster than one CTA with twice the pipeline depth.
static int g_stages = 6, g_ctas_per_sm = 2;
static int g_split_penalty_pm = 10;  // cost of one more k split, per mille of the streaming time (see choose_split)
static int g_l2_next_every = 4;      // see tc_set_l2_prefetch: every n-th k block of the announced GEMM goes to L2 early (0 = off)
constexpr unsigned long long kWaitCycles = 3000000000ull;   // ~1.5 s at 2 GHz

struct alignas(64) TcParams {
    CUtensorMap tmA[3];
    CUtensorMap tmB;
    int n_mats;
    int chunk_end[3];   // cumulative slab counts
    int n_rows[3];      // rows of each matrix
    int n_off[3];       // first output column of each matrix
    int n_chunks, R, S, KB, n_items;
    int stages;
    // L2 prefetch on behalf of a later (pair mode) GEMM whose weights this kernel's idle wait can hide
    CUtensorMap tmN[2];
    int next_half, next_chunks, next_KB, next_every;   // next_every = 0: none
    float* out;
    int n_total;
    int r0, m;
    // gate/up pair mode: every work item is half gate rows (tile rows 0 ..), half up rows (tile rows 64 ..)
    int pair_half;              // rows of each kind per item (<= 64)
    __nv_bfloat16* swiglu_out;  // [16][n_rows[0]]: high halves in rows 0-7, low halves in rows 8-15
    // LM-head mode
    float inv_tau, threshold;
    float* conf;
    int* token;
    int* exit_flag;
    float* logits_dbg;
    SoftTriple* part;
    unsigned int* ticket;
    unsigned int* status;
    Mirror mirror;
};

struct TcPlan {
    TcParams p;
    int grid;
};

void TcPlanCache::clear() {
    for (auto& kv : plans) delete kv.second;
    plans.clear();
}

// ---------------------------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------------------------
// Bounded wait.  Returns false (and raises the abort flag + status word) if the budget runs out
// or another role of this CTA already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, unsigned int* status,
                                          unsigned int code, unsigned long long budget = kWaitCycles) {
    if (mbar_try_wait(bar, parity)) return true;
    unsigned long long t0 = clock64();
    for (;;) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > budget) {
            *abort_flag = 1;
            atomicExch(status, code);
            return false;
        }
    }
}
// Same, for waits that are expected to last long (an epilogue warp waiting for a whole work
// item): backs off with nanosleep so that the polling does not compete with the producers.
__device__ __forceinline__ bool mbar_wait_relaxed(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                                  unsigned int* status, unsigned int code) {
    if (mbar_try_wait(bar, parity)) return true;
    unsigned long long t0 = clock64();
    for (;;) {
        __nanosleep(200);
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > kWaitCycles) {
            *abort_flag = 1;
            atomicExch(status, code);
            return false;
        }
    }
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* tm, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
        "l"(tm), "r"(x), "r"(y), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void tma_load_2d_hint(uint32_t dst, const CUtensorMap* tm, int x, int y, uint32_t bar,
                                                 uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], "
        "[%4], %5;" ::"r"(dst),
        "l"(tm), "r"(x), "r"(y), "r"(bar), "l"(policy)
        : "memory");
}
__device__ __forceinline__ uint64_t policy_evict_first() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d),
        "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void tc_ld16(uint32_t taddr, uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
// shared-memory matrix descriptor: K-major operand, 128-byte swizzle, 8-row groups 1024 bytes apart
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr) {
    uint64_t d = (uint64_t)((addr & 0x3ffffu) >> 4);
    d |= (uint64_t)1 << 16;              // leading byte offset (unused for swizzled K-major): 16 bytes
    d |= (uint64_t)(1024 >> 4) << 32;    // stride byte offset between 8-row groups
    d |= (uint64_t)1 << 46;              // descriptor version of sm_100
    d |= (uint64_t)2 << 61;              // SWIZZLE_128B
    return d;
}
// instruction descriptor: D = f32, A = B = bf16, both K-major, N columns (16 per block of 8 activation rows), M = 128
__host__ __device__ constexpr uint32_t idesc_n(uint32_t n) { return (1u << 4) | (1u << 7) | (1u << 10) | ((n >> 3) << 17) | ((128u >> 4) << 24); }

// The four epilogue warps agree on whether to go on: each has waited (bounded) for the accumulator on its
// own, and a named barrier that one of them skipped would hang the others.  ok_s is [2][4], alternating per call.
__device__ __forceinline__ bool epi_vote(bool ok, volatile int* ok_s, int n_call, int q, int lane) {
    volatile int* slot = ok_s + (n_call & 1) * 4;
    if (lane == 0) slot[q] = ok ? 1 : 0;
    asm volatile("bar.sync 1, 128;" ::: "memory");
    return (slot[0] & slot[1] & slot[2] & slot[3]) != 0;
}

struct ItemInfo {
    int mat, row0, kb0, kb1;
};
__device__ __forceinline__ ItemInfo decode_item(const TcParams& p, int item) {
    int chunk = item % p.n_chunks, s = item / p.n_chunks;
    if (p.pair_half) return ItemInfo{0, chunk * p.pair_half, 0, p.KB};   // never split along k
    int j = 0, base = 0;
    while (j < p.n_mats - 1 && chunk >= p.chunk_end[j]) base = p.chunk_end[j++];
    ItemInfo it;
    it.mat = j;
    it.row0 = (chunk - base) * p.R;
    it.kb0 = (int)((long long)s * p.KB / p.S);
    it.kb1 = (int)((long long)(s + 1) * p.KB / p.S);
    return it;
}

// Position of a CTA in its sequence of (work item, k block) pipeline fills.
struct WorkIter {
    int item, kb;
    ItemInfo it;
    __device__ explicit WorkIter(const TcParams& p) : item((int)blockIdx.x), kb(0) {
        if (valid_item(p)) { it = decode_item(p, item); kb = it.kb0; }
        n_items = p.n_items;
    }
    int n_items;
    __device__ bool valid_item(const TcParams& p) const { return item < p.n_items; }
    __device__ bool valid() const { return item < n_items; }
    __device__ void next(const TcParams& p) {
        if (item >= n_items) return;
        if (++kb < it.kb1) return;
        item += (int)gridDim.x;
        if (item < p.n_items) { it = decode_item(p, item); kb = it.kb0; }
    }
};

template <bool kHead, bool kPair, int NB = 1>
__global__ void __launch_bounds__(kTcThreads, 2) k_tc(const __grid_constant__ TcParams p) {
    static_assert(!kHead || NB == 1, "the LM-head mode handles one block of rows");
    constexpr int kStageBn = NB * kStageB;          // activation tile of a stage: 16 operand rows per block
    constexpr uint32_t kCols = 16u * NB;            // TMEM columns of one accumulator
    constexpr uint32_t kIdesc = idesc_n(kCols);
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint32_t tmem_base_s;
    __shared__ volatile int abort_s;
    __shared__ SoftTriple cta_part[4][kMaxW];
    __shared__ bool is_last_s;
    __shared__ float up_s[kPair ? kMaxW * 64 : 1];   // pair mode: the up projections of an item, [row][column in item]
    __shared__ volatile int ok_s[8];

    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles = (raw + 1023u) & ~1023u;             // swizzled tiles need 1024-byte alignment
    const int kStages = p.stages;
    const uint32_t smA = tiles, smB = tiles + kStages * kStageA;
    const uint32_t bars = smB + kStages * kStageBn;            // 8-byte mbarriers
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (kStages + s); };
    auto tfull_bar = [&](int b) { return bars + 8u * (2 * kStages + b); };
    auto tempty_bar = [&](int b) { return bars + 8u * (2 * kStages + 2 + b); };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    pdl_trigger();
    if (threadIdx.x == 0) {
        abort_s = 0;
        for (int s = 0; s < kStages; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(tfull_bar(b), 1);
            mbar_init(tempty_bar(b), 4);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kProducers) {   // TMEM: two accumulators of 16 columns per block of rows
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(2u * kCols));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_s;
    const uint32_t stage_bytes = (uint32_t)p.R * (kBK * 2) + kStageBn;

    if (warp < kProducers) {
        // ------------------------------ TMA producers ------------------------------
        // Producer j owns pipeline fills j, j + kProducers, ...  The weight tiles of the first
        // pipeline fill do not depend on the preceding kernel, so they are requested BEFORE the
        // grid-dependency wait; the activation tiles (written by that kernel) follow after it.
        if (lane == 0) {
            if (warp == 0) {
                for (int j = 0; j < p.n_mats; ++j) asm volatile("prefetch.tensormap [%0];" ::"l"(&p.tmA[j]) : "memory");
                asm volatile("prefetch.tensormap [%0];" ::"l"(&p.tmB) : "memory");
            }
            const uint64_t pol = policy_evict_first();
            // weight tile(s) of one pipeline fill; pair mode: gate rows to tile rows 0 .., up rows to tile rows 64 ..
            auto load_a = [&](int st, const WorkIter& wi) {
                if (kPair) {
                    tma_load_2d_hint(smA + st * kStageA, &p.tmA[0], wi.kb * kBK, wi.it.row0, full_bar(st), pol);
                    tma_load_2d_hint(smA + st * kStageA + 64 * kBK * 2, &p.tmA[1], wi.kb * kBK, wi.it.row0, full_bar(st), pol);
                } else {
                    tma_load_2d_hint(smA + st * kStageA, &p.tmA[wi.it.mat], wi.kb * kBK, wi.it.row0, full_bar(st), pol);
                }
            };
            WorkIter w(p), w0(p);
            for (int j = 0; j < warp; ++j) { w.next(p); w0.next(p); }
            int fill = warp;
            for (; w.valid() && fill < kStages; fill += kProducers) {
                mbar_expect_tx(full_bar(fill), stage_bytes);
                load_a(fill, w);
                for (int j = 0; j < kProducers; ++j) w.next(p);
            }
            // Still waiting for the predecessor kernel, and so will the kernels after this one: HBM would
            // sit idle.  Ask TMA to bring every next_every-th k block of the weights of a GEMM that runs
            // later into L2 (no shared memory, no barrier involved), so that it then streams from L2 and
            // HBM side by side.
            if (p.next_every > 0) {
                for (int c = blockIdx.x; c < p.next_chunks; c += gridDim.x)
                    for (int kb = warp * p.next_every; kb < p.next_KB; kb += kProducers * p.next_every) {
                        asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global [%0, {%1, %2}];" ::"l"(&p.tmN[0]), "r"(kb * kBK),
                                     "r"(c * p.next_half)
                                     : "memory");
                        asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global [%0, {%1, %2}];" ::"l"(&p.tmN[1]), "r"(kb * kBK),
                                     "r"(c * p.next_half)
                                     : "memory");
                    }
            }
            pdl_wait();
            for (int f0 = warp; f0 < fill; f0 += kProducers) {
                tma_load_2d(smB + f0 * kStageBn, &p.tmB, w0.kb * kBK, 0, full_bar(f0));
                for (int j = 0; j < kProducers; ++j) w0.next(p);
            }
            for (; w.valid(); fill += kProducers) {
                int stage = fill % kStages;
                uint32_t phase = (uint32_t)(fill / kStages) & 1u;
                if (!mbar_wait(empty_bar(stage), phase ^ 1u, &abort_s, p.status, 1u)) break;
                mbar_expect_tx(full_bar(stage), stage_bytes);
                load_a(stage, w);
                tma_load_2d(smB + stage * kStageBn, &p.tmB, w.kb * kBK, 0, full_bar(stage));
                for (int j = 0; j < kProducers; ++j) w.next(p);
            }
        } else {
            pdl_wait();
        }
    } else if (warp == kProducers) {
        // ------------------------------ MMA issuer ------------------------------
        pdl_wait();
        if (lane == 0) {
            int stage = 0, phase = 0, n_local = 0;
            bool ok = true;
            for (int item = blockIdx.x; item < p.n_items && ok; item += gridDim.x, ++n_local) {
                ItemInfo it = decode_item(p, item);
                int buf = n_local & 1;
                uint32_t use = (uint32_t)(n_local >> 1);   // how often this accumulator was used before
                if (!(ok = mbar_wait(tempty_bar(buf), (use & 1u) ^ 1u, &abort_s, p.status, 2u))) break;
                tc_fence_after();
                uint32_t d_tmem = tmem_base + (uint32_t)buf * kCols;
                for (int kb = it.kb0; kb < it.kb1; ++kb) {
                    if (!(ok = mbar_wait(full_bar(stage), phase, &abort_s, p.status, 3u))) break;
                    tc_fence_after();
                    uint64_t da = smem_desc(smA + stage * kStageA), db = smem_desc(smB + stage * kStageBn);
#pragma unroll
                    for (int k = 0; k < kBK / 16; ++k)   // +32 bytes per 16-element k step inside the swizzle row
                        tc_mma(d_tmem, da + 2u * k, db + 2u * k, kIdesc, (kb > it.kb0 || k > 0) ? 1u : 0u);
                    tc_commit(empty_bar(stage));          // frees the stage once these MMAs have read it
                    if (++stage == kStages) { stage = 0; phase ^= 1; }
                }
                if (ok) tc_commit(tfull_bar(buf));        // accumulator complete
            }
        }
    } else {
        // ------------------------------ epilogue (128 threads) ------------------------------
        pdl_wait();
        const int q = warp & 3;                            // TMEM lane quadrant this warp may read
        const int row_in_tile = q * 32 + lane;
        SoftTriple tr[kMaxW];
        if (kHead) {
#pragma unroll
            for (int i = 0; i < kMaxW; ++i) tr[i] = soft_empty();
        }
        int n_local = 0;
        bool ok = true;
        for (int item = blockIdx.x; item < p.n_items && ok; item += gridDim.x, ++n_local) {
            ItemInfo it = decode_item(p, item);
            int buf = n_local & 1;
            uint32_t use = (uint32_t)(n_local >> 1);
            if (lane == 0) ok = mbar_wait_relaxed(tfull_bar(buf), use & 1u, &abort_s, p.status, 4u);
            ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;   // one lane polls; the TMEM load needs the whole warp
            if (kPair) ok = epi_vote(ok, ok_s, n_local, q, lane);   // the pair epilogue synchronises the four warps
            if (!ok) break;
            tc_fence_after();
            for (int blk = 0; blk < NB; ++blk) {           // one block of 8 activation rows = 16 accumulator columns
                uint32_t v[16];
                tc_ld16(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)buf * kCols + (uint32_t)blk * 16u, v);
                if (blk == NB - 1) {
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(tempty_bar(buf));   // accumulator may be overwritten
                }
                const int row_base = blk * kMaxW;          // first activation row of this block
                if (kPair) {
                    // warps 2-3 hold the up projections (tile rows 64 ..): hand them to the thread that holds the
                    // gate projection of the same column, which writes silu(gate) * up as the next GEMM's operand
                    float z[kMaxW];
#pragma unroll
                    for (int i = 0; i < kMaxW; ++i) z[i] = __uint_as_float(v[i]) + __uint_as_float(v[i + 8]);
                    if (q >= 2) {
#pragma unroll
                        for (int i = 0; i < kMaxW; ++i) up_s[i * 64 + (row_in_tile - 64)] = z[i];
                    }
                    asm volatile("bar.sync 1, 128;" ::: "memory");
                    const int col = it.row0 + row_in_tile;
                    if (q < 2 && row_in_tile < p.pair_half && col < p.n_rows[0]) {
                        const size_t F = (size_t)p.n_rows[0];
                        __nv_bfloat16* dst = p.swiglu_out + (size_t)blk * 16 * F;   // [16][F] per block: high halves, low halves
#pragma unroll
                        for (int i = 0; i < kMaxW; ++i) {
                            if (row_base + i >= p.r0 && row_base + i < p.r0 + p.m) {
                                const float g = z[i], u = up_s[i * 64 + row_in_tile];
                                const float val = g / (1.f + expf(-g)) * u;
                                const __nv_bfloat16 hi = __float2bfloat16_rn(val);
                                dst[(size_t)i * F + col] = hi;
                                dst[(size_t)(i + 8) * F + col] = __float2bfloat16_rn(val - __bfloat162float(hi));
                            }
                        }
                    }
                    asm volatile("bar.sync 1, 128;" ::: "memory");   // up_s may be overwritten by the next block / item
                    continue;
                }
                const int n = it.row0 + row_in_tile;
                if (row_in_tile < p.R && n < p.n_rows[it.mat]) {
                    const int s = item / p.n_chunks;
#pragma unroll
                    for (int i = 0; i < kMaxW; ++i) {
                        if (row_base + i >= p.r0 && row_base + i < p.r0 + p.m) {
                            float z = __uint_as_float(v[i]) + __uint_as_float(v[i + 8]);
                            if (kHead) {
                                soft_push(tr[i], z, n, p.inv_tau);
                                if (p.logits_dbg) p.logits_dbg[(size_t)(i - p.r0) * p.n_total + n] = z;
                            } else {   // split-K partials [block][split][8][n_total]
                                p.out[(((size_t)blk * p.S + s) * kMaxW + i) * p.n_total + p.n_off[it.mat] + n] = z;
                            }
                        }
                    }
                }
            }
        }
        if (kHead) {
            // lanes -> warp: butterfly merge (both partners compute the same merged triple)
#pragma unroll
            for (int i = 0; i < kMaxW; ++i) {
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    SoftTriple other;
                    other.m = __shfl_xor_sync(0xffffffffu, tr[i].m, o);
                    other.idx = __shfl_xor_sync(0xffffffffu, tr[i].idx, o);
                    other.s = __shfl_xor_sync(0xffffffffu, tr[i].s, o);
                    tr[i] = soft_merge(tr[i], other, p.inv_tau);
                }
                if (lane == 0) cta_part[q][i] = tr[i];
            }
        }
    }

    if (abort_s) {   // a wait expired: give copies and MMAs still in flight time to land before leaving
        unsigned long long t0 = clock64();
        while (clock64() - t0 < 4000000ull) {}
    }
    tc_fence_before();
    __syncthreads();
    if (warp == kProducers) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(2u * kCols));
    }
    if (!kHead) return;

    // CTA triples -> scratch; the last CTA to arrive merges all CTAs in index order (wait-free)
    if (threadIdx.x < kMaxW) {
        int i = threadIdx.x;
        SoftTriple t = cta_part[0][i];
        for (int w = 1; w < 4; ++w) t = soft_merge(t, cta_part[w][i], p.inv_tau);
        p.part[(size_t)blockIdx.x * kMaxW + i] = t;
        __threadfence();
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned int prev = atomicAdd(p.ticket, 1u);
        is_last_s = (prev == gridDim.x - 1);
    }
    __syncthreads();
    if (!is_last_s) return;
    __threadfence();
    soft_final_merge(p.part, (int)gridDim.x, p.r0, p.m, p.inv_tau, p.threshold, p.conf, p.token, p.exit_flag);
    if (threadIdx.x == 0) *p.ticket = 0u;
    publish_results(p.mirror);
}

// ---------------------------------------------------------------------------------------------
// Wide passes (prefill, 128 activation rows) on CTA PAIRS: tcgen05.mma.cta_group::2, M = 256, N = 16 .. 256.
//
// At 128 rows the pass is bound by the tensor pipe, so the operands swap roles against the 8-row kernel: the
// ACTIVATIONS are the MMA's M operand (256 operand rows = 128 rows x high/low halves; each CTA of the pair holds 128 of
// them = 64 rows, and accumulates them in its own tensor memory), the WEIGHT rows of a work item are the N operand
// (2 R rows, R of them staged by each CTA), and N can be any multiple of 16: the host picks the tile width that
// spreads a matrix evenly over the clusters (gate/up of the 7B shape: 22016 rows are 1.16 rounds of 128-row tiles,
// i.e. 2 rounds at 62 % fill with weights as M; as N they are two rounds of 160 columns).  Measured, a k block costs a
// cluster the same 0.34-0.38 us at every width tried (at N = 256 that is the measured tensor peak), so the decomposition
// prefers wide tiles and few k blocks per cluster.  Both CTAs stage their operand halves with plain TMA copies, each into its own shared memory; the
// MMA, issued by one thread of the first CTA, reads both halves out of both CTAs' shared memory.
//
// Accumulator of a CTA: lane = operand row (block b = lanes 16 b .. 16 b + 15: high halves of rows 8 b .. 8 b + 7, then
// their low halves), column = weight row of the item.  The epilogue adds the low half's lane to the high half's with
// a shuffle and writes 16-byte pieces.  Gate/up: the first CTA stages the item's gate rows, the second its up rows,
// so a lane holds gate (columns 0 .. h-1) and up (columns h .. 2 h - 1) of the same output and applies SwiGLU itself.
//
// Barriers: "full" lives in the first CTA (the leader) and counts the bytes of BOTH CTAs' copies (each CTA issues its
// own copies with the pair form of the instruction, which may complete on the peer's barrier); "stage empty" and
// "accumulator full" exist in both CTAs and are signalled together by the leader's tcgen05.commit; "accumulator
// empty" lives in the leader and takes the arrivals of both CTAs' epilogue warps.  Every wait is bounded as in k_tc.
// ---------------------------------------------------------------------------------------------
constexpr int kPairStages = 6;
constexpr int kStageB2 = 128 * kBK * 2;       // this CTA's half of the activation tile: 16 KB
constexpr uint32_t kPairCols = 256;           // TMEM columns of one accumulator (16 per block of 8 rows)
static int smem_bytes_pair() { return kPairStages * (kStageA + kStageB2) + 1024 + 256; }
static_assert(kPairStages * (kStageA + kStageB2) + 1280 + 16384 + 512 <= 227 * 1024, "pair stages exceed shared memory");
// D = f32, A = B = bf16, both K-major, M = 256 (the pair), N columns
__host__ __device__ constexpr uint32_t idesc_pair(uint32_t n) { return (1u << 4) | (1u << 7) | (1u << 10) | ((n >> 3) << 17) | ((256u >> 4) << 24); }

__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void cluster_sync_pair() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// pair form of the TMA tile copy: destination in this CTA, completion on a barrier of either CTA of the pair
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* tm, int x, int y, uint32_t bar_cluster, uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], "
        "[%4], %5;" ::"r"(dst),
        "l"(tm), "r"(x), "r"(y), "r"(bar_cluster), "l"(policy)
        : "memory");
}
__device__ __forceinline__ uint64_t policy_evict_last() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ void tc_mma_pair(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d),
        "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
        : "memory");
}
// completion of the MMAs issued so far arrives on the barrier at this shared-memory offset in BOTH CTAs of the pair
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {
    const uint16_t both = 3;
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar), "h"(both)
                 : "memory");
}

// 64 consecutive accumulator columns of this warp's 32 lanes (no wait: pair with tc_wait_ld)
__device__ __forceinline__ void tc_ld64_nowait(uint32_t taddr, uint32_t (&v)[64]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x64.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32, %33, %34, %35, %36, %37, %38, %39, %40, %41, %42, %43, %44, %45, %46, %47, %48, %49, %50, %51, %52, %53, %54, %55, %56, %57, %58, %59, %60, %61, %62, %63}, [%64];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31]), "=r"(v[32]), "=r"(v[33]), "=r"(v[34]), "=r"(v[35]), "=r"(v[36]), "=r"(v[37]), "=r"(v[38]), "=r"(v[39]), "=r"(v[40]), "=r"(v[41]), "=r"(v[42]), "=r"(v[43]), "=r"(v[44]), "=r"(v[45]), "=r"(v[46]), "=r"(v[47]), "=r"(v[48]), "=r"(v[49]), "=r"(v[50]), "=r"(v[51]), "=r"(v[52]), "=r"(v[53]), "=r"(v[54]), "=r"(v[55]), "=r"(v[56]), "=r"(v[57]), "=r"(v[58]), "=r"(v[59]), "=r"(v[60]), "=r"(v[61]), "=r"(v[62]), "=r"(v[63])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tc_ld32_nowait(uint32_t taddr, uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Work items of the pair kernel: (slab of 2 R weight rows, k split); CTA r of the pair stages rows row0 + r R ..
// (gate/up: the h columns row0 .. of the gate matrix for r = 0, of the up matrix for r = 1).  Clusters stride over
// the items.  first_row: the first weight row (output column) of the item.
__device__ __forceinline__ ItemInfo decode_item_pair(const TcParams& p, int item, int rank, int* first_row) {
    ItemInfo it = decode_item(p, item);
    if (p.pair_half) {
        it.row0 = (item % p.n_chunks) * p.pair_half;
        *first_row = it.row0;
    } else {
        *first_row = 2 * it.row0;                  // decode_item counted slabs of R rows; a pair slab is 2 R
        it.row0 = 2 * it.row0 + rank * p.R;
    }
    return it;
}

template <bool kPair>
__global__ void __launch_bounds__(kTcThreads, 1) k_tc_pair(const __grid_constant__ TcParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint32_t tmem_base_s;
    __shared__ volatile int abort_s;

    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles = (raw + 1023u) & ~1023u;
    constexpr int kStages = kPairStages;
    const uint32_t smA = tiles, smB = tiles + kStages * kStageA;
    const uint32_t bars = smB + kStages * kStageB2;
    auto full_bar = [&](int s) { return bars + 8u * s; };                       // used in the leader
    auto empty_bar = [&](int s) { return bars + 8u * (kStages + s); };          // both CTAs
    auto tfull_bar = [&](int b) { return bars + 8u * (2 * kStages + b); };      // both CTAs
    auto tempty_bar = [&](int b) { return bars + 8u * (2 * kStages + 2 + b); }; // used in the leader

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_rank();
    const int cluster_id = (int)(blockIdx.x >> 1), n_clusters = (int)(gridDim.x >> 1);   // clusters of two CTAs along x (the pair of a 2-CTA MMA)
    pdl_trigger();
    if (threadIdx.x == 0) {
        abort_s = 0;
        for (int s = 0; s < kStages; ++s) {
            mbar_init(full_bar(s), 1);       // the leader's arrive.expect_tx; the bytes of both CTAs
            mbar_init(empty_bar(s), 1);      // the leader's commit
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(tfull_bar(b), 1);      // the leader's commit
            mbar_init(tempty_bar(b), 8);     // four epilogue warps of each CTA
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kProducers) {   // both accumulators of both CTAs: the same warp of each CTA takes part
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(2u * kPairCols));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::);
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_pair();        // the peer's barriers exist before anything arrives on them
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_s;
    const int R = kPair ? p.pair_half : p.R;                             // weight rows this CTA stages per fill
    const uint32_t stage_bytes = 2u * ((uint32_t)R * (kBK * 2) + (uint32_t)kStageB2);   // what both CTAs bring per fill

    if (warp < kProducers) {
        // ------------------------------ TMA producers (both CTAs) ------------------------------
        if (lane == 0) {
            if (warp == 0) {
                for (int j = 0; j < p.n_mats; ++j) asm volatile("prefetch.tensormap [%0];" ::"l"(&p.tmA[j]) : "memory");
                asm volatile("prefetch.tensormap [%0];" ::"l"(&p.tmB) : "memory");
            }
            const uint64_t pol_w = policy_evict_first(), pol_a = policy_evict_last();
            // position in this cluster's sequence of (item, k block) fills
            int item = cluster_id, kb = 0;
            ItemInfo it{};
            int first_row_unused = 0;
            auto start_item = [&]() { if (item < p.n_items) { it = decode_item_pair(p, item, (int)rank, &first_row_unused); kb = it.kb0; } };
            auto advance = [&]() {
                if (item >= p.n_items) return;
                if (++kb < it.kb1) return;
                item += n_clusters;
                start_item();
            };
            start_item();
            for (int j = 0; j < warp; ++j) advance();
            auto load_a = [&](int st, uint32_t bar) {   // this CTA's weight rows (gate/up: the first CTA's are gate rows, the second's up rows)
                tma_load_2d_pair(smA + st * kStageA, &p.tmA[kPair ? (int)rank : it.mat], kb * kBK, it.row0, bar, pol_w);
            };
            // The weight tiles of the first pipeline fill do not depend on the preceding kernel: requested before the
            // grid-dependency wait; the activation tiles follow after it.
            int fill = warp;
            int kb_first[(kStages + kProducers - 1) / kProducers];
            int n_first = 0;
            for (; item < p.n_items && fill < kStages; fill += kProducers) {
                if (rank == 0) mbar_expect_tx(full_bar(fill), stage_bytes);
                load_a(fill, map_to_cta(full_bar(fill), 0));
                kb_first[n_first++] = kb;
                for (int j = 0; j < kProducers; ++j) advance();
            }
            pdl_wait();
            for (int j = 0; j < n_first; ++j) {
                const int f0 = warp + j * kProducers;
                tma_load_2d_pair(smB + f0 * kStageB2, &p.tmB, kb_first[j] * kBK, 128 * (int)rank, map_to_cta(full_bar(f0), 0), pol_a);
            }
            for (; item < p.n_items; fill += kProducers) {
                const int stage = fill % kStages;
                const uint32_t phase = (uint32_t)(fill / kStages) & 1u;
                if (!mbar_wait(empty_bar(stage), phase ^ 1u, &abort_s, p.status, 1u)) break;
                if (rank == 0) mbar_expect_tx(full_bar(stage), stage_bytes);
                const uint32_t bar = map_to_cta(full_bar(stage), 0);
                load_a(stage, bar);
                tma_load_2d_pair(smB + stage * kStageB2, &p.tmB, kb * kBK, 128 * (int)rank, bar, pol_a);
                for (int j = 0; j < kProducers; ++j) advance();
            }
        } else {
            pdl_wait();
        }
    } else if (warp == kProducers) {
        // ------------------------------ MMA issuer (one thread of the leader) ------------------------------
        pdl_wait();
        if (rank == 0 && lane == 0) {
            const uint32_t idesc = idesc_pair(2u * (uint32_t)R);
            int stage = 0, phase = 0, n_local = 0;
            bool ok = true;
            for (int item = cluster_id; item < p.n_items && ok; item += n_clusters, ++n_local) {
                const ItemInfo it = decode_item(p, item);
                const int buf = n_local & 1;
                const uint32_t use = (uint32_t)(n_local >> 1);
                if (!(ok = mbar_wait(tempty_bar(buf), (use & 1u) ^ 1u, &abort_s, p.status, 2u))) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)buf * kPairCols;
                for (int kb = it.kb0; kb < it.kb1; ++kb) {
                    if (!(ok = mbar_wait(full_bar(stage), phase, &abort_s, p.status, 3u))) break;
                    tc_fence_after();
                    // A = the activation halves (M), B = the weight rows (N)
                    const uint64_t da = smem_desc(smB + stage * kStageB2), db = smem_desc(smA + stage * kStageA);
#pragma unroll
                    for (int k = 0; k < kBK / 16; ++k)
                        tc_mma_pair(d_tmem, da + 2u * k, db + 2u * k, idesc, (kb > it.kb0 || k > 0) ? 1u : 0u);
                    tc_commit_pair(empty_bar(stage));     // frees the stage in both CTAs once these MMAs have read it
                    if (++stage == kStages) { stage = 0; phase ^= 1; }
                }
                if (ok) tc_commit_pair(tfull_bar(buf));   // accumulators of both CTAs complete
            }
        }
    } else {
        // ------------------------------ epilogue (128 threads of each CTA) ------------------------------
        // An item's main loop is short at 128 rows (a few microseconds), so the epilogue must be short too: tensor-memory
        // loads of 32-64 columns, the next one in flight while the current one is stored, and compact code (a loop,
        // not thousands of straight-line instructions that would all be instruction-cache misses).
        pdl_wait();
        const int q = warp & 3;
        const int o = 128 * (int)rank + 32 * q + lane;      // operand row of this lane
        const int blk = o >> 4, i_row = o & 7;              // block of 8 rows, row in the block
        const int row = blk * kMaxW + i_row;
        const bool row_ok = (o & 8) == 0 && row >= p.r0 && row < p.r0 + p.m;   // high-half lanes store; lane + 8 holds the low half
        const int N = 2 * R;
        int n_local = 0;
        bool ok = true;
        for (int item = cluster_id; item < p.n_items && ok; item += n_clusters, ++n_local) {
            int first_row = 0;
            const ItemInfo it = decode_item_pair(p, item, (int)rank, &first_row);
            const int buf = n_local & 1;
            const uint32_t use = (uint32_t)(n_local >> 1);
            if (lane == 0) ok = mbar_wait_relaxed(tfull_bar(buf), use & 1u, &abort_s, p.status, 4u);
            ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
            if (!ok) break;
            tc_fence_after();
            const uint32_t t0 = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)buf * kPairCols;
            if constexpr (kPair) {
                // columns 0 .. h-1: gate projections, h .. 2 h - 1: up projections of FFN columns first_row ..
                const int h = R, F = p.n_rows[0];
                __nv_bfloat16* dst = p.swiglu_out + ((size_t)blk * 16 + i_row) * F + first_row;   // high halves; low halves 8 rows on
                uint32_t g[32], u[32];
#pragma unroll 1
                for (int c0 = 0; c0 < h; c0 += 32) {
                    tc_ld32_nowait(t0 + (uint32_t)c0, g);
                    tc_ld32_nowait(t0 + (uint32_t)(h + c0), u);
                    tc_wait_ld();
#pragma unroll
                    for (int c8 = 0; c8 < 4; ++c8) {
                        uint32_t hi[4], lo[4];
#pragma unroll
                        for (int c2 = 0; c2 < 4; ++c2) {
                            float val[2];
#pragma unroll
                            for (int e = 0; e < 2; ++e) {
                                const int c = c8 * 8 + c2 * 2 + e;
                                const float gh = __uint_as_float(g[c]), uh = __uint_as_float(u[c]);
                                const float gt = gh + __shfl_down_sync(0xffffffffu, gh, 8), up = uh + __shfl_down_sync(0xffffffffu, uh, 8);
                                val[e] = __fdividef(gt, 1.f + __expf(-gt)) * up;   // fast exponential and division: this epilogue is a chain of dependent instructions on one warp per scheduler
                            }
                            const __nv_bfloat162 vh = __floats2bfloat162_rn(val[0], val[1]);
                            const __nv_bfloat162 vl = __floats2bfloat162_rn(val[0] - __bfloat162float(vh.x), val[1] - __bfloat162float(vh.y));
                            hi[c2] = *reinterpret_cast<const uint32_t*>(&vh);
                            lo[c2] = *reinterpret_cast<const uint32_t*>(&vl);
                        }
                        const int c = c0 + c8 * 8;
                        if (row_ok && c < h && first_row + c < F) {     // h and F are multiples of 8: a piece is all in or all out
                            *reinterpret_cast<uint4*>(dst + c) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
                            *reinterpret_cast<uint4*>(dst + (size_t)8 * F + c) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
                        }
                    }
                }
            } else {
                // partials [block][split][8][n_total]; columns first_row .. first_row + N - 1 of matrix it.mat
                const int s = item / p.n_chunks;
                float* orow = p.out + (((size_t)blk * p.S + s) * kMaxW + i_row) * p.n_total + p.n_off[it.mat] + first_row;
                const int n_lim = min(N, p.n_rows[it.mat] - first_row);
                auto finish_group = [&](int c0, const uint32_t (&v)[64]) {
#pragma unroll
                    for (int c4 = 0; c4 < 16; ++c4) {
                        float x[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const float hi = __uint_as_float(v[c4 * 4 + e]);
                            x[e] = hi + __shfl_down_sync(0xffffffffu, hi, 8);
                        }
                        const int c = c0 + c4 * 4;
                        if (row_ok && c < n_lim) {
                            if (c + 3 < n_lim) {
                                *reinterpret_cast<float4*>(orow + c) = make_float4(x[0], x[1], x[2], x[3]);
                            } else {
#pragma unroll
                                for (int e = 0; e < 4; ++e)
                                    if (c + e < n_lim) orow[c + e] = x[e];
                            }
                        }
                    }
                };
                uint32_t va[64], vb[64];
                tc_ld64_nowait(t0, va);
#pragma unroll 1
                for (int c0 = 0; c0 < N; c0 += 128) {     // two groups of 64 columns per trip: one register buffer each
                    tc_wait_ld();
                    if (c0 + 64 < N) tc_ld64_nowait(t0 + (uint32_t)(c0 + 64), vb);
                    finish_group(c0, va);
                    if (c0 + 64 < N) {
                        tc_wait_ld();
                        if (c0 + 128 < N) tc_ld64_nowait(t0 + (uint32_t)(c0 + 128), va);
                        finish_group(c0 + 64, vb);
                    }
                }
            }
            // every load of this accumulator has completed: it may be overwritten
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(map_to_cta(tempty_bar(buf), 0));
        }
    }

    if (abort_s) {   // a wait expired: give copies and MMAs still in flight time to land before leaving
        unsigned long long t0 = clock64();
        while (clock64() - t0 < 4000000ull) {}
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_pair();   // neither CTA's shared memory, barriers or tensor memory go away while the peer may still use them
    if (warp == kProducers) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(2u * kPairCols));
    }
}

// ---------------------------------------------------------------------------------------------
// Host side: tensor maps and work decomposition
// ---------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
        else
            (void)cudaGetLastError();
    }
    return fn;
}

bool tc_available() { return true; }

static bool make_map(CUtensorMap* tm, const void* base, int rows, int K, int box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)K * 2};
    cuuint32_t box[2] = {(cuuint32_t)kBK, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

static int sm_count() { return device_sm_count(); }

// Slab height R (multiple of 8 in [64,128]) and split count S that minimise what the busiest
// CTA streams.  Depends on the shape only, never on the number of rows.
static void choose_split(const int* n_rows, int n_mats, int KB, int max_split, int G, int* R_out, int* S_out) {
    double best = 1e300;
    int bR = 128, bS = 1;
    for (int S = 1; S <= max_split && S <= KB; ++S)
        for (int R = 128; R >= 64; R -= 8) {
            long long chunks = 0;
            for (int j = 0; j < n_mats; ++j) chunks += (n_rows[j] + R - 1) / R;
            long long items = chunks * S;
            long long per = (items + G - 1) / G;
            double cost = (double)per * R * ((KB + S - 1) / S) * (1.0 + 0.001 * g_split_penalty_pm * S);   // each split adds partial traffic and consumer loads
            if (cost < best - 1e-9) { best = cost; bR = R; bS = S; }
        }
    *R_out = bR;
    *S_out = bS;
}

// Pair mode: rows of each kind per item (multiple of 8 in [32,64]) that minimise what the busiest CTA streams.
static int choose_pair_half(int n_rows, int G) {
    double best = 1e300;
    int bh = 64;
    for (int h = 64; h >= 32; h -= 8) {
        long long items = (n_rows + h - 1) / h;
        double cost = (double)((items + G - 1) / G) * h;
        if (cost < best - 1e-9) { best = cost; bh = h; }
    }
    return bh;
}

// Work decomposition of the CTA-pair kernel: R (multiple of 8, <= 128) and the split count that minimise what the
// busiest cluster spends.  G = clusters.  Measured: a k block costs a cluster 0.34-0.38 us whatever the tile width
// (N = 112, 160, 176 or 256 columns; at 256 that is the measured tensor peak, and 4 stages instead of 6 cost 5 % only),
// so narrow tiles buy nothing below ~96 rows per CTA: the cost of an item is charged as if it had at least
// that many (floor 32 / 64 / 96 / 128: 512-token prefill 22.4 / 20.2 / 20.0 / 20.4 ms).
static int g_pair_floor_rows = 96, g_pair_split_pm = 30;
static void choose_split_cta_pair(const int* n_rows, int n_mats, int KB, int max_split, int G, int* R_out, int* S_out) {
    double best = 1e300;
    int bR = 128, bS = 1;
    for (int S = 1; S <= max_split && S <= KB; ++S)
        for (int R = 128; R >= 8; R -= 8) {
            long long chunks = 0;
            for (int j = 0; j < n_mats; ++j) chunks += (n_rows[j] + 2 * R - 1) / (2 * R);
            const long long per = (chunks * S + G - 1) / G;
            const double cost = (double)per * (R > g_pair_floor_rows ? R : g_pair_floor_rows) * ((KB + S - 1) / S) *
                                (1.0 + 0.001 * g_pair_split_pm * (S - 1));
            if (cost < best - 1e-9) { best = cost; bR = R; bS = S; }
        }
    *R_out = bR;
    *S_out = bS;
}
// gate/up: FFN columns per item (the first CTA stages that many gate rows, the second as many up rows; never split along k)
static int choose_cols_cta_pair(int n_rows, int G) {
    double best = 1e300;
    int bh = 128;
    for (int h = 128; h >= 8; h -= 8) {
        const long long items = (n_rows + h - 1) / h;
        const double cost = (double)((items + G - 1) / G) * (h > g_pair_floor_rows ? h : g_pair_floor_rows);
        if (cost < best - 1e-9) { best = cost; bh = h; }
    }
    return bh;
}

static int max_pair_clusters();
// cta_pair: plan for k_tc_pair (a work item is a slab of 2 R rows for a cluster of two CTAs)
static TcPlan* get_plan(TcPlanCache* cache, const void* const* W, const int* n_end, int n_mats, int K, const void* act,
                        bool head, bool pair = false, int nb = 1, bool cta_pair = false) {
    std::vector<uint64_t> key;
    for (int j = 0; j < n_mats; ++j) { key.push_back((uint64_t)(uintptr_t)W[j]); key.push_back((uint64_t)n_end[j]); }
    key.push_back((uint64_t)K);
    key.push_back((uint64_t)(uintptr_t)act);
    key.push_back((head ? 1 : 0) + (pair ? 2 : 0) + 4 * nb + (cta_pair ? 1024 : 0));
    key.push_back((uint64_t)g_stages * 16 + g_ctas_per_sm + ((uint64_t)g_split_penalty_pm << 40));
    auto it = cache->plans.find(key);
    if (it != cache->plans.end()) return it->second;
    TcPlan* pl = new TcPlan();
    memset(&pl->p, 0, sizeof(pl->p));
    TcParams& p = pl->p;
    int G = cta_pair ? max_pair_clusters() : sm_count() * (nb > 1 ? 1 : g_ctas_per_sm);   // CTAs, or clusters, that share the items
    if (G > sm_count() / 2 && cta_pair) G = sm_count() / 2;
    p.stages = cta_pair ? kPairStages : nb > 1 ? kWideStages : g_stages;
    p.n_mats = n_mats;
    p.KB = (K + kBK - 1) / kBK;
    int prev = 0;
    for (int j = 0; j < n_mats; ++j) { p.n_rows[j] = n_end[j] - prev; p.n_off[j] = prev; prev = n_end[j]; }
    int chunks = 0;
    const int per_item = cta_pair ? 2 : 1;   // CTAs that share a work item
    if (pair && cta_pair) {
        p.pair_half = choose_cols_cta_pair(p.n_rows[0], G);
        p.R = p.pair_half;
        p.S = 1;
        chunks = (p.n_rows[0] + p.pair_half - 1) / p.pair_half;
        for (int j = 0; j < 3; ++j) p.chunk_end[j] = chunks;
    } else if (pair) {
        p.pair_half = choose_pair_half(p.n_rows[0], G);
        p.R = 2 * p.pair_half;
        p.S = 1;
        chunks = (p.n_rows[0] + p.pair_half - 1) / p.pair_half;
        for (int j = 0; j < 3; ++j) p.chunk_end[j] = chunks;
    } else {
        if (cta_pair) choose_split_cta_pair(p.n_rows, n_mats, p.KB, kMaxSplit, G, &p.R, &p.S);
        else choose_split(p.n_rows, n_mats, p.KB, head ? 1 : kMaxSplit, G, &p.R, &p.S);
        for (int j = 0; j < 3; ++j) {
            if (j < n_mats) chunks += (p.n_rows[j] + per_item * p.R - 1) / (per_item * p.R);
            p.chunk_end[j] = chunks;
        }
    }
    p.n_chunks = chunks;
    p.n_items = chunks * p.S;
    pl->grid = (p.n_items < G ? p.n_items : G) * per_item;
    bool ok = make_map(&p.tmB, act, 16 * nb, K, cta_pair ? 128 : 16 * nb);
    for (int j = 0; j < n_mats && ok; ++j) ok = make_map(&p.tmA[j], W[j], p.n_rows[j], K, pair ? p.pair_half : p.R);
    if (!ok) { delete pl; return nullptr; }
    cache->plans[key] = pl;
    return pl;
}

// The decomposition the launches use, for a given number of CTAs (8-row kernel) or clusters (CTA-pair kernel): host
// arithmetic only.  mode 0: 8-row kernel, 1: its gate/up form, 2: 128-row CTA-pair kernel, 3: its gate/up form.
bool tc_plan_query(int mode, const int* n_rows, int n_mats, int K, int units, int* R, int* S, int* n_items) {
    if (mode < 0 || mode > 3 || !n_rows || n_mats < 1 || n_mats > 3 || K < 1 || units < 1) return false;
    for (int j = 0; j < n_mats; ++j)
        if (n_rows[j] < 1) return false;
    const int KB = (K + kBK - 1) / kBK;
    if (mode == 1 || mode == 3) {
        const int h = mode == 3 ? choose_cols_cta_pair(n_rows[0], units) : choose_pair_half(n_rows[0], units);
        *R = h; *S = 1; *n_items = (n_rows[0] + h - 1) / h;
        return true;
    }
    if (mode == 2) choose_split_cta_pair(n_rows, n_mats, KB, kMaxSplit, units, R, S);
    else choose_split(n_rows, n_mats, KB, kMaxSplit, units, R, S);
    const int per = mode == 2 ? 2 : 1;
    int chunks = 0;
    for (int j = 0; j < n_mats; ++j) chunks += (n_rows[j] + per * *R - 1) / (per * *R);
    *n_items = chunks * *S;
    return true;
}

template <bool kHead, bool kPair, int NB = 1> static void launch(cudaStream_t st, const TcPlan* pl, const TcParams& p) {
    static bool attr_set[kMaxDevices];   // function attributes are per device
    const int dev = current_device();
    if (dev >= 0 && !attr_set[dev]) {
        cudaFuncSetAttribute(k_tc<kHead, kPair, NB>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             NB > 1 ? smem_bytes(kWideStages, NB) : smem_bytes(kMaxStages));
        attr_set[dev] = true;
    }
    launch_k(k_tc<kHead, kPair, NB>, dim3(pl->grid), dim3(kTcThreads), (size_t)smem_bytes(p.stages, NB), st, p);
}

template <bool kPair> static void pair_func_attr() {
    static bool attr_set[kMaxDevices];
    const int dev = current_device();
    if (dev >= 0 && !attr_set[dev]) {
        cudaFuncSetAttribute(k_tc_pair<kPair>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes_pair());
        attr_set[dev] = true;
    }
}
template <bool kPair> static bool launch_pair(cudaStream_t st, const TcPlan* pl, const TcParams& p) {
    pair_func_attr<kPair>();
    const bool ok = launch_kcp(k_tc_pair<kPair>, dim3(pl->grid), dim3(kTcThreads), (size_t)smem_bytes_pair(), st, dim3(2, 1, 1), g_use_pdl, p) == cudaSuccess;
    if (!ok && getenv("SB_DEBUG")) fprintf(stderr, "[specbound] k_tc_pair: grid %d, smem %d, items %d, clusters at once %d\n", pl->grid, smem_bytes_pair(), p.n_items, max_pair_clusters());
    return ok;
}
// Clusters of two k_tc_pair CTAs the device can hold at once (a GPC with an odd number of usable SMs leaves one out):
// the persistent grid must not exceed it, or the last cluster would run as a second wave.  0 = cannot run.
static int max_pair_clusters() {
    static int n[kMaxDevices];   // 0 unknown, -1 none
    const int dev = current_device();
    if (dev < 0) return 0;
    if (n[dev] == 0) {
        pair_func_attr<false>();
        cudaLaunchConfig_t cfg{};
        cfg.gridDim = dim3((unsigned)(sm_count() / 2 * 2)); cfg.blockDim = dim3(kTcThreads); cfg.dynamicSmemBytes = (size_t)smem_bytes_pair();
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeClusterDimension;
        at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
        cfg.attrs = at; cfg.numAttrs = 1;
        int c = 0;
        if (cudaOccupancyMaxActiveClusters(&c, k_tc_pair<false>, &cfg) != cudaSuccess) { (void)cudaGetLastError(); c = 0; }
        n[dev] = c > 0 ? c : -1;
    }
    return n[dev] > 0 ? n[dev] : 0;
}

static bool g_wide_cta_pairs = true;   // wide passes on CTA pairs (k_tc_pair) instead of single CTAs (k_tc<., ., 16>)
void tc_set_wide_cta_pairs(bool on) { g_wide_cta_pairs = on; }

bool tc_set_split_penalty(int per_mille) {
    if (per_mille < 0 || per_mille > 1000) return false;
    g_split_penalty_pm = per_mille;
    return true;
}

bool tc_set_l2_prefetch(int every) {
    if (every < 0 || every > 64) return false;
    g_l2_next_every = every;
    return true;
}

// Self-test of the bounded wait: one CTA waits on an mbarrier that nothing ever completes, with a
// small cycle budget.  The wait must give up, raise the status word and let the kernel return.
__global__ void k_wait_selftest(unsigned int* status, unsigned long long budget_cycles, unsigned int* waited_flag) {
    __shared__ __align__(8) unsigned long long bar;
    __shared__ volatile int abort_s;
    if (threadIdx.x == 0) {
        abort_s = 0;
        mbar_init(smem_u32(&bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        bool ok = mbar_wait(smem_u32(&bar), 0, &abort_s, status, 9u, budget_cycles);
        *waited_flag = ok ? 1u : 2u;
    }
}
void launch_wait_selftest(cudaStream_t st, unsigned int* status, unsigned long long budget_cycles, unsigned int* waited_flag) {
    k_wait_selftest<<<1, 32, 0, st>>>(status, budget_cycles, waited_flag);
}

bool tc_set_tuning(int stages, int ctas_per_sm) {
    // stages >= producers: a producer's parity wait on a stage's "empty" barrier is only sound if no
    // peer can lag two phases behind, which in-order consumption guarantees when stages >= producers
    if (stages < kProducers || stages > kMaxStages || ctas_per_sm < 1 || ctas_per_sm > 2) return false;
    if (ctas_per_sm * (smem_bytes(stages) + 2048) > 227 * 1024) return false;
    g_stages = stages;
    g_ctas_per_sm = ctas_per_sm;
    return true;
}

int launch_gemm_tc(cudaStream_t st, const GemmArgs& a, TcPlanCache* cache, unsigned int* status) {
    const bool pair = a.swiglu_out != nullptr;
    if (pair && (a.n_mats != 2 || a.n_end[1] != 2 * a.n_end[0])) return -1;
    const int nb = a.nb > 1 ? kWideBlocks : 1;
    if (a.nb > 1 && a.nb != kWideBlocks) return -1;
    const bool cta_pair = nb > 1 && g_wide_cta_pairs && max_pair_clusters() > 0;
    TcPlan* pl = get_plan(cache, a.W, a.n_end, a.n_mats, a.K, a.act, false, pair, nb, cta_pair);
    if (!pl) return -1;
    TcParams p = pl->p;
    p.out = a.out; p.n_total = a.n_total; p.r0 = a.r0; p.m = a.m; p.status = status;
    if (cta_pair) {
        if (pair) {
            p.swiglu_out = reinterpret_cast<__nv_bfloat16*>(a.swiglu_out);
            if (!launch_pair<true>(st, pl, p)) return -1;
        } else {
            if (!launch_pair<false>(st, pl, p)) return -1;
        }
        return p.S;
    }
    if (a.next_W[0] && g_l2_next_every > 0 && nb == 1) {   // announce a later pair-mode GEMM: same plan that GEMM will use
        const void* nW[2] = {a.next_W[0], a.next_W[1]};
        int n_end[2] = {a.next_rows, 2 * a.next_rows};
        TcPlan* nx = get_plan(cache, nW, n_end, 2, a.next_K, a.next_act, false, true);
        if (nx) {
            p.tmN[0] = nx->p.tmA[0]; p.tmN[1] = nx->p.tmA[1];
            p.next_half = nx->p.pair_half; p.next_chunks = nx->p.n_chunks; p.next_KB = nx->p.KB;
            p.next_every = g_l2_next_every;
        }
    }
    if (pair) {
        p.swiglu_out = reinterpret_cast<__nv_bfloat16*>(a.swiglu_out);
        if (nb > 1) launch<false, true, kWideBlocks>(st, pl, p);
        else launch<false, true>(st, pl, p);
    } else {
        if (nb > 1) launch<false, false, kWideBlocks>(st, pl, p);
        else launch<false, false>(st, pl, p);
    }
    return p.S;
}

bool launch_head_tc(cudaStream_t st, const HeadArgs& a, TcPlanCache* cache, unsigned int* status) {
    const void* W[1] = {a.W};
    int n_end[1] = {a.V};
    TcPlan* pl = get_plan(cache, W, n_end, 1, a.K, a.act, true);
    if (!pl) return false;
    TcParams p = pl->p;
    p.n_total = a.V; p.r0 = a.r0; p.m = a.m; p.status = status;
    p.inv_tau = a.inv_tau; p.threshold = a.threshold; p.conf = a.conf; p.token = a.token; p.exit_flag = a.exit_flag;
    p.logits_dbg = a.logits_dbg; p.part = a.part; p.ticket = a.ticket; p.mirror = a.mirror;
    launch<true, false>(st, pl, p);
    return true;
}

}  // namespace sb
