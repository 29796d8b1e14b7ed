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

static TcPlan* get_plan(TcPlanCache* cache, const void* const* W, const int* n_end, int n_mats, int K, const void* act,
                        bool head, bool pair = false, int nb = 1) {
    std::vector<uint64_t> key;
    for (int j = 0; j < n_mats; ++j) { key.push_back((uint64_t)(uintptr_t)W[j]); key.push_back((uint64_t)n_end[j]); }
    key.push_back((uint64_t)K);
    key.push_back((uint64_t)(uintptr_t)act);
    key.push_back((head ? 1 : 0) + (pair ? 2 : 0) + 4 * nb);
    key.push_back((uint64_t)g_stages * 16 + g_ctas_per_sm + ((uint64_t)g_split_penalty_pm << 40));
    auto it = cache->plans.find(key);
    if (it != cache->plans.end()) return it->second;
    TcPlan* pl = new TcPlan();
    memset(&pl->p, 0, sizeof(pl->p));
    TcParams& p = pl->p;
    int G = sm_count() * (nb > 1 ? 1 : g_ctas_per_sm);
    p.stages = nb > 1 ? kWideStages : g_stages;
    p.n_mats = n_mats;
    p.KB = (K + kBK - 1) / kBK;
    int prev = 0;
    for (int j = 0; j < n_mats; ++j) { p.n_rows[j] = n_end[j] - prev; p.n_off[j] = prev; prev = n_end[j]; }
    int chunks = 0;
    if (pair) {
        p.pair_half = choose_pair_half(p.n_rows[0], G);
        p.R = 2 * p.pair_half;
        p.S = 1;
        chunks = (p.n_rows[0] + p.pair_half - 1) / p.pair_half;
        for (int j = 0; j < 3; ++j) p.chunk_end[j] = chunks;
    } else {
        choose_split(p.n_rows, n_mats, p.KB, head ? 1 : kMaxSplit, G, &p.R, &p.S);
        for (int j = 0; j < 3; ++j) {
            if (j < n_mats) chunks += (p.n_rows[j] + p.R - 1) / p.R;
            p.chunk_end[j] = chunks;
        }
    }
    p.n_chunks = chunks;
    p.n_items = chunks * p.S;
    pl->grid = p.n_items < G ? p.n_items : G;
    bool ok = make_map(&p.tmB, act, 16 * nb, K, 16 * nb);
    for (int j = 0; j < n_mats && ok; ++j) ok = make_map(&p.tmA[j], W[j], p.n_rows[j], K, pair ? p.pair_half : p.R);
    if (!ok) { delete pl; return nullptr; }
    cache->plans[key] = pl;
    return pl;
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
    TcPlan* pl = get_plan(cache, a.W, a.n_end, a.n_mats, a.K, a.act, false, pair, nb);
    if (!pl) return -1;
    TcParams p = pl->p;
    p.out = a.out; p.n_total = a.n_total; p.r0 = a.r0; p.m = a.m; p.status = status;
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
