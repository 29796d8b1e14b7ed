// Host side of the SpecBound library: context, workspace layout, the layer step, the round loop
// of Section 3.3 and the C ABI declared in include/specbound.h.  Every arithmetic step runs in a
// kernel; the host only sequences launches and reads the few integers that gate the next launch
// (exit flag after a probe, acceptance count after a round).
#include <chrono>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>

#include "gemm_tc.cuh"
#include "sb_internal.cuh"

namespace sb {

static int g_default_gemm = -1;   // -1: pick tcgen05 for bf16 when available
static int g_fuse = 3;            // bit 0: SwiGLU in the epilogue of the tcgen05 gate/up GEMM; bit 1: RoPE + append + attention + chunk merge in one launch
static int g_wide_prefill = 1;    // prefill: up to 128 prompt rows per pass of the weight-streaming GEMMs (bf16, tcgen05 path)
static int g_qkv_ahead = 1;       // draft loop: issue the next layer step's norm + QKV GEMM while waiting for the exit decision
static int g_trace = 0;           // 1: the stateless layer call times every launch with CUDA events and prints them

// TMA descriptors of the stateless entry points: keyed by (pointers, shapes), so they stay valid for as
// long as the key matches; kept across calls because encoding them costs more host time than the launch.
// One cache per device (a descriptor holds a device address and the plan the device's SM count); the stateless
// entry points hold g_stateless_mu while they use it, so they may be called from several host threads.
static std::mutex g_stateless_mu;
static TcPlanCache& stateless_plans() {
    static TcPlanCache cache[kMaxDevices];
    int dev = current_device();
    TcPlanCache& c = cache[dev < 0 ? 0 : dev];
    if (c.plans.size() > 512) c.clear();
    return c;
}

struct Tracer {
    static constexpr int kMax = 64;
    cudaEvent_t ev[kMax];
    const char* name[kMax];
    int n = 0;
    bool on = false;
    cudaStream_t st;
    void begin(cudaStream_t s) {
        on = true; st = s; n = 0;
        mark("start");
    }
    void mark(const char* what) {
        if (!on || n >= kMax) return;
        cudaEventCreate(&ev[n]);
        cudaEventRecord(ev[n], st);
        name[n++] = what;
    }
    void end() {
        if (!on) return;
        cudaEventSynchronize(ev[n - 1]);
        float tot = 0.f;
        cudaEventElapsedTime(&tot, ev[0], ev[n - 1]);
        fprintf(stderr, "[sb trace] %d launches, %.1f us:", n - 1, tot * 1e3f);
        for (int i = 1; i < n; ++i) {
            float ms = 0.f;
            cudaEventElapsedTime(&ms, ev[i - 1], ev[i]);
            fprintf(stderr, " %s=%.1f", name[i], ms * 1e3f);
        }
        fprintf(stderr, "\n");
        for (int i = 0; i < n; ++i) cudaEventDestroy(ev[i]);
        on = false;
    }
};
static Tracer g_tracer;
#define SB_MARK(what) g_tracer.mark(what)

struct Dims {
    int L, d, H, Hkv, hd, F, V, qd, kvd;
    int page, page_shift, n_pages, max_seq, chunk;
    float rope_base, eps;
    bool f32;
    double inv_freq[64];
};

static int pick_gemm(bool f32) {
    if (f32 || !tc_available()) return 0;
    return g_default_gemm < 0 ? 1 : g_default_gemm;
}

static bool is_pow2(int v) { return v > 0 && (v & (v - 1)) == 0; }

static bool make_dims(const sb_config* c, Dims* o) {
    if (!c) return false;
    if (c->n_layers < 1 || c->n_layers > SB_MAX_LAYERS || c->d_model < 8 || c->n_heads < 1 || c->n_kv_heads < 1 ||
        c->d_ffn < 8 || c->vocab < 2 || c->max_seq < 1)
        return false;
    if (c->n_heads % c->n_kv_heads) return false;
    // the attention kernels keep all (row, query head) pairs of a KV head in one CTA's shared memory: 8 rows x 4 heads
    if (c->n_heads / c->n_kv_heads > 4) return false;
    if (c->head_dim != 32 && c->head_dim != 64 && c->head_dim != 128) return false;
    if (c->d_model % 8 || c->d_ffn % 8 || c->d_model > 8192) return false;
    if (c->dtype != SB_F32 && c->dtype != SB_BF16) return false;
    if (!is_pow2(c->kv_page) || c->kv_page < 16) return false;
    if (!(c->rope_base > 0.f) || !(c->rms_eps > 0.f)) return false;
    o->L = c->n_layers; o->d = c->d_model; o->H = c->n_heads; o->Hkv = c->n_kv_heads; o->hd = c->head_dim;
    o->F = c->d_ffn; o->V = c->vocab; o->qd = o->H * o->hd; o->kvd = o->Hkv * o->hd;
    o->page = c->kv_page; o->page_shift = 0;
    while ((1 << o->page_shift) < o->page) ++o->page_shift;
    o->max_seq = c->max_seq;
    o->n_pages = (c->max_seq + o->page - 1) / o->page;
    // split-KV chunk: fixed per context so that a row's attention never depends on its companions
    o->chunk = 128;   // = the attention kernel's chunk: 4 warps x 32 positions
    o->rope_base = c->rope_base; o->eps = c->rms_eps; o->f32 = c->dtype == SB_F32;
    for (int i = 0; i < o->hd / 2; ++i) o->inv_freq[i] = std::pow((double)c->rope_base, -2.0 * i / o->hd);
    return true;
}

constexpr int kWideRows = kWideBlocks * kMaxW;   // rows of one wide prefill pass

// Scratch shared by the context and the stateless entry points.
struct Work {
    int* page_table;
    float* h;              // [8][d] hidden-state cache: one vector per in-flight row
    void *act_a, *act_b, *act_o, *act_f;   // act_b: the hidden rows under a second norm (layer_step's next_gain2)
    float *p_qkv, *p_o, *p_gu, *p_down;   // split-K partials [kMaxSplit][8][N]
    float* q;              // [8][qd]
    float* attn_part;
    SoftTriple* head_part;
    unsigned int* ticket;
    int* res;              // result block: conf[8] | token[8] | flag[8] | accept[10] (32-bit words)
    int* toks;             // [max_seq + 8] device token log
    unsigned int* status;  // device status word of the bounded waits
    float2* rope_tab;      // contexts only: cos/sin of the RoPE angles [n_pages * page][hd/2]
    float* logits;         // contexts only: [8][V] final logits of the rows being sampled (sampling decoding)
    double* sample_e;      // contexts only: [8][V] their exponentials
    // contexts of bf16 models only: the wide prefill pass (kWideBlocks = B blocks of 8 rows per launch of the GEMMs)
    float* pf_h;           // [8 B][d]
    void *pf_act_a, *pf_act_o, *pf_act_f;      // [B][16][d | qd | F]
    float *pf_p_qkv, *pf_p_o, *pf_p_down;      // [B][kMaxSplit][8][N]
    float *pf_q, *pf_attn_part;                // [8 B][qd]; [B][max_chunks][8][H][hd+2]
    size_t pf_attn_stride;                     // floats per block of pf_attn_part
    unsigned long long* sample_q;   // contexts only: [8][V] the same as fixed-point integers (top-p)
    void* k_cache;         // [L][n_pages][page][kvd]
    void* v_cache;
};

struct Carver {
    char* base;
    size_t off = 0;
    template <typename P> void take(P*& p, size_t bytes) {
        off = (off + 1023) & ~size_t(1023);
        p = reinterpret_cast<P*>(base ? base + off : nullptr);
        off += bytes;
    }
};

static size_t carve(const Dims& D, char* base, bool with_state, Work* w) {
    Carver c{base};
    Work tmp;
    Work& W = w ? *w : tmp;
    size_t es = D.f32 ? 4 : 2, act_rows = D.f32 ? 8 : 16;
    c.take(W.page_table, sizeof(int) * D.n_pages);
    c.take(W.h, sizeof(float) * kMaxW * D.d);
    c.take(W.act_a, es * act_rows * D.d);
    c.take(W.act_b, es * act_rows * D.d);
    c.take(W.act_o, es * act_rows * D.qd);
    c.take(W.act_f, es * act_rows * D.F);
    size_t ps = sizeof(float) * kMaxSplit * kMaxW;
    c.take(W.p_qkv, ps * (D.qd + 2 * D.kvd));
    c.take(W.p_o, ps * D.d);
    c.take(W.p_gu, ps * 2 * D.F);
    c.take(W.p_down, ps * D.d);
    c.take(W.q, sizeof(float) * kMaxW * D.qd);
    int max_chunks = (D.max_seq + kMaxW + D.chunk - 1) / D.chunk + 1;
    c.take(W.attn_part, sizeof(float) * (size_t)max_chunks * kMaxW * D.H * (D.hd + 2));
    c.take(W.head_part, sizeof(SoftTriple) * kHeadMaxCtas * kMaxW);
    c.take(W.res, sizeof(int) * 64);
    // the status word sits inside the result block (word 48), so that one copy brings results and status to the host;
    // the exit kernel's ticket follows (word 56): one 64-byte clear resets both
    W.status = reinterpret_cast<unsigned int*>(W.res + 48);
    W.ticket = reinterpret_cast<unsigned int*>(W.res + 56);
    W.rope_tab = nullptr;
    W.logits = nullptr;
    W.sample_e = nullptr;
    W.sample_q = nullptr;
    W.pf_h = nullptr;
    if (with_state) {
        c.take(W.toks, sizeof(int) * (D.max_seq + 16));
        c.take(W.logits, sizeof(float) * (size_t)kMaxW * D.V);
        c.take(W.sample_e, sizeof(double) * (size_t)kMaxW * D.V);
        c.take(W.sample_q, sizeof(unsigned long long) * (size_t)kMaxW * D.V);
        if (!D.f32) {
            c.take(W.pf_h, sizeof(float) * kWideRows * D.d);
            c.take(W.pf_act_a, es * 2 * kWideRows * D.d);
            c.take(W.pf_act_o, es * 2 * kWideRows * D.qd);
            c.take(W.pf_act_f, es * 2 * kWideRows * D.F);
            const size_t pw = sizeof(float) * kMaxSplit * kWideRows;
            c.take(W.pf_p_qkv, pw * (D.qd + 2 * D.kvd));
            c.take(W.pf_p_o, pw * D.d);
            c.take(W.pf_p_down, pw * D.d);
            c.take(W.pf_q, sizeof(float) * kWideRows * D.qd);
            W.pf_attn_stride = (size_t)max_chunks * kMaxW * D.H * (D.hd + 2);
            c.take(W.pf_attn_part, sizeof(float) * kWideBlocks * W.pf_attn_stride);
        }
        c.take(W.rope_tab, sizeof(float2) * (size_t)D.n_pages * D.page * (D.hd / 2));
        size_t kv = es * (size_t)D.L * D.n_pages * D.page * D.kvd;
        c.take(W.k_cache, kv);
        c.take(W.v_cache, kv);
    }
    return (c.off + 1023) & ~size_t(1023);
}

struct Exec {   // everything a launch sequence needs
    Dims D;
    Work W;
    cudaStream_t st;
    int gemm;   // 0 simt, 1 tcgen05
    int64_t launches = 0;
    // which normalised activation act_a currently holds
    const void* act_gain = nullptr;
    int act_r0 = 0, act_m = 0;
    const void* act2_gain = nullptr;      // ... and act_b (same rows), null = nothing valid
    TcPlanCache* plans = nullptr;
    unsigned int* clear_next = nullptr;   // 16 words that the next RMSNorm launch of ensure_act zeroes (stateless calls)
    int err = 0;   // sticky host-side error of a launch sequence (a TMA descriptor could not be built)
};

#define SB_T(E, call)                          \
    do {                                       \
        if ((E).D.f32) { using T = float; call; } \
        else { using T = __nv_bfloat16; call; }   \
    } while (0)

static void ensure_act(Exec& e, const void* gain, int r0, int m) {
    if (e.act_gain == gain && r0 >= e.act_r0 && r0 + m <= e.act_r0 + e.act_m) return;
    SB_T(e, launch_resid_norm<T>(e.st, e.W.h, nullptr, 0, e.D.d, (const T*)gain, e.D.eps, e.W.act_a, r0, m, e.clear_next));
    e.clear_next = nullptr;
    e.launches++;
    if (r0 != e.act_r0 || m != e.act_m) e.act2_gain = nullptr;   // the row range describes both buffers
    e.act_gain = gain; e.act_r0 = r0; e.act_m = m;
}

// out = act x W^T for up to three matrices; returns the number of split-K partials written
static bool tc_path(const Exec& e) { return e.gemm == 1 && !e.D.f32; }
struct NextGemm { const void* W[2] = {nullptr, nullptr}; int rows = 0, K = 0; const void* act = nullptr; };
static int gemm(Exec& e, const void* const* W, const int* N, int n_mats, int K, const void* act, float* out, int r0, int m,
                void* swiglu_out = nullptr, const NextGemm& next = NextGemm(), int nb = 1) {
    GemmArgs a{};
    a.nb = nb;
    a.swiglu_out = swiglu_out;
    a.next_W[0] = next.W[0]; a.next_W[1] = next.W[1]; a.next_rows = next.rows; a.next_K = next.K; a.next_act = next.act;
    int tot = 0;
    for (int j = 0; j < n_mats; ++j) { a.W[j] = W[j]; tot += N[j]; a.n_end[j] = tot; }
    for (int j = n_mats; j < 3; ++j) { a.W[j] = nullptr; a.n_end[j] = 0x7fffffff; }
    a.n_mats = n_mats; a.K = K; a.act = act; a.out = out; a.n_total = tot; a.r0 = r0; a.m = m;
    e.launches++;
    if (e.gemm == 1 && !e.D.f32) {
        int s = launch_gemm_tc(e.st, a, e.plans, e.W.status);
        if (s < 1) { e.err = SB_ERR_CUDA; return 1; }
        return s;
    }
    SB_T(e, launch_gemm_simt<T>(e.st, a));
    return 1;
}

// One decoder layer for rows r0 .. r0+m-1 (row i sits at position pos0 + i).  Ends by adding the
// MLP output to the hidden rows and, if next_gain is given, leaving their RMSNorm in act_a.
// The first two launches of a layer step: RMSNorm of the rows with the layer's attention gain (if the operand does
// not hold it already) and the QKV GEMM.  They read the hidden rows and write scratch only, so the draft loop may
// issue them ahead of time (qkv_ahead) while the host still waits for an exit decision.  Returns the split count.
static int layer_qkv(Exec& e, const sb_layer_weights& lw, int r0, int m) {
    const Dims& D = e.D;
    // the step that produced these rows may have left them under this layer's norm in the second operand buffer (it
    // knew that an exit test would take the first): no RMSNorm launch then
    const bool second = e.act2_gain == lw.attn_norm && e.act_gain != lw.attn_norm && r0 >= e.act_r0 && r0 + m <= e.act_r0 + e.act_m;
    if (!second) ensure_act(e, lw.attn_norm, r0, m);
    const void* wqkv[3] = {lw.wq, lw.wk, lw.wv};
    int nqkv[3] = {D.qd, D.kvd, D.kvd};
    SB_MARK("norm");
    int s_qkv = gemm(e, wqkv, nqkv, 3, D.d, second ? e.W.act_b : e.W.act_a, e.W.p_qkv, r0, m);
    SB_MARK("qkv");
    return s_qkv;
}

// s_qkv_ahead > 0: layer_qkv was already issued for exactly these rows of this layer, with that split count
// next_gain2 (nullable): a second gain under which the rows' RMSNorm is left as well (in act_b)
static void layer_step(Exec& e, const sb_layer_weights& lw, void* k_cache_l, void* v_cache_l, int r0, int m, int pos0,
                       const void* next_gain, int s_qkv_ahead = 0, const void* next_gain2 = nullptr) {
    const Dims& D = e.D;
    Work& W = e.W;
    const int s_qkv = s_qkv_ahead > 0 ? s_qkv_ahead : layer_qkv(e, lw, r0, m);
    AttnArgs aa{W.q, k_cache_l, v_cache_l, W.page_table, W.attn_part, W.act_o, D.H, D.Hkv, D.hd, D.page, D.page_shift,
                pos0, r0, m, D.chunk, W.p_qkv, s_qkv, W.rope_tab, W.status, {}};
    for (int i = 0; i < D.hd / 2; ++i) aa.inv_freq[i] = D.inv_freq[i];
    bool fused = false;
    if (g_fuse & 2) SB_T(e, fused = launch_attention_fused<T>(e.st, aa));   // RoPE + append + attention + merge in one launch
    if (fused) {
        e.launches += 1;
        SB_MARK("attn");
    } else {
        // more than 8 chunks: the chunk kernel with the same front end, then the chunk merge (two launches)
        bool front = false;
        if (g_fuse & 2) SB_T(e, front = launch_attention_front<T>(e.st, aa));
        if (front) {
            e.launches += 2;
            SB_MARK("attn");
        } else {
            RopeArgs ra{W.p_qkv, s_qkv, W.q, k_cache_l, v_cache_l, W.page_table, D.H, D.Hkv, D.hd, D.page, D.page_shift,
                        pos0, r0, m, D.rope_base, W.rope_tab, {}};
            for (int i = 0; i < D.hd / 2; ++i) ra.inv_freq[i] = D.inv_freq[i];
            SB_T(e, launch_rope_append<T>(e.st, ra));
            SB_MARK("rope");
            bool ok = false;
            SB_T(e, ok = launch_attention<T>(e.st, aa));
            if (!ok) e.err = SB_ERR_UNSUPPORTED;
            SB_MARK("attn");
            e.launches += 3;
        }
    }
    const void* wo[1] = {lw.wo};
    int no[1] = {D.d};
    // the output projection waits through the whole attention chain with HBM idle: it announces the
    // gate/up GEMM so that part of those weights is already in L2 when their turn comes
    NextGemm nx;
    if (tc_path(e) && (g_fuse & 1)) { nx.W[0] = lw.w_gate; nx.W[1] = lw.w_up; nx.rows = D.F; nx.K = D.d; nx.act = W.act_a; }
    int s_o = gemm(e, wo, no, 1, D.qd, W.act_o, W.p_o, r0, m, nullptr, nx);
    SB_MARK("o");
    SB_T(e, launch_resid_norm<T>(e.st, W.h, W.p_o, s_o, D.d, (const T*)lw.mlp_norm, D.eps, W.act_a, r0, m));
    SB_MARK("norm2");
    const void* wgu[2] = {lw.w_gate, lw.w_up};
    int ngu[2] = {D.F, D.F};
    if (tc_path(e) && (g_fuse & 1)) {   // SwiGLU in the gate/up GEMM's epilogue: act_f comes straight out of it
        gemm(e, wgu, ngu, 2, D.d, W.act_a, W.p_gu, r0, m, W.act_f);
        SB_MARK("gateup");
    } else {
        int s_gu = gemm(e, wgu, ngu, 2, D.d, W.act_a, W.p_gu, r0, m);
        SB_MARK("gateup");
        SB_T(e, launch_swiglu<T>(e.st, W.p_gu, s_gu, D.F, W.act_f, r0, m));
        e.launches++;
        SB_MARK("swiglu");
    }
    const void* wd[1] = {lw.w_down};
    int nd[1] = {D.d};
    int s_d = gemm(e, wd, nd, 1, D.F, W.act_f, W.p_down, r0, m);
    SB_MARK("down");
    if (!next_gain) next_gain2 = nullptr;
    SB_T(e, launch_resid_norm<T>(e.st, W.h, W.p_down, s_d, D.d, (const T*)next_gain, D.eps, W.act_a, r0, m, nullptr,
                                 (const T*)next_gain2, W.act_b));
    SB_MARK("resid");
    e.launches += 2;
    e.act_gain = next_gain; e.act_r0 = r0; e.act_m = m;
    e.act2_gain = next_gain2;
}

// Wide prefill pass: one decoder layer for M <= 8 * kWideBlocks prompt rows at positions pos0 .. pos0+M-1 (bf16
// models, tcgen05 GEMMs with the SwiGLU epilogue).  The four weight-streaming GEMMs take all rows in ONE launch each
// (blocks of 8 rows: the weights are read once for 128 rows instead of once for 8); so do the residual/RMSNorm
// kernel and the RoPE/append kernel; the attention kernels run all full blocks in one launch (a block per grid.z),
// after the append, so that a block's attention sees the K/V rows of the blocks before it.  have_act: pf_act_a
// already holds the rows' RMSNorm with this layer's attention gain (left there by the previous layer).  Ends by
// adding the MLP output to pf_h and, if next_gain is given, leaving the rows' RMSNorm with that gain in pf_act_a.
static void layer_step_wide(Exec& e, const sb_layer_weights& lw, void* k_cache_l, void* v_cache_l, int M, int pos0,
                            bool have_act, const void* next_gain) {
    using T = __nv_bfloat16;
    const Dims& D = e.D;
    Work& W = e.W;
    auto act_of = [&](void* base, int b, int K) { return (void*)((char*)base + (size_t)b * 16 * K * sizeof(T)); };
    if (!have_act) {
        launch_resid_norm<T>(e.st, W.pf_h, nullptr, 0, D.d, (const T*)lw.attn_norm, D.eps, W.pf_act_a, 0, M);
        e.launches++;
    }
    const void* wqkv[3] = {lw.wq, lw.wk, lw.wv};
    int nqkv[3] = {D.qd, D.kvd, D.kvd};
    const int s_qkv = gemm(e, wqkv, nqkv, 3, D.d, W.pf_act_a, W.pf_p_qkv, 0, M, nullptr, NextGemm(), kWideBlocks);
    // RoPE + K/V append for all rows in one launch, then the separate attention kernels over all full blocks of 8
    // rows at once (grid.z = block; every block sees the K/V rows of the blocks before it, already appended), then
    // the ragged last block, if any, by itself
    {
        RopeArgs ra{W.pf_p_qkv, s_qkv, W.pf_q, k_cache_l, v_cache_l, W.page_table, D.H, D.Hkv, D.hd, D.page, D.page_shift,
                    pos0, 0, M, D.rope_base, W.rope_tab, {}};
        for (int i = 0; i < D.hd / 2; ++i) ra.inv_freq[i] = D.inv_freq[i];
        launch_rope_append<T>(e.st, ra);
        e.launches++;
        const int n_full = M / kMaxW, rem = M - n_full * kMaxW;
        // tiled causal attention on the tensor cores: one launch for all rows of the pass
        bool tiled = false;
        if (g_wide_prefill != 2 && (D.hd == 64 || D.hd == 128))
            tiled = launch_attention_prefill(e.st, W.pf_q, k_cache_l, v_cache_l, W.page_table, W.pf_act_o, D.H, D.Hkv, D.hd, D.page,
                                             D.page_shift, pos0, M);
        if (tiled) e.launches++;
        if (!tiled && n_full > 0) {
            AttnArgs aa{W.pf_q, k_cache_l, v_cache_l, W.page_table, W.pf_attn_part, W.pf_act_o, D.H, D.Hkv, D.hd, D.page,
                        D.page_shift, pos0, 0, kMaxW, D.chunk, nullptr, 0, W.rope_tab, W.status, {}};
            aa.n_blocks = n_full;
            aa.part_block_stride = W.pf_attn_stride;
            aa.pos_pred0 = pos0;
            if (!launch_attention<T>(e.st, aa)) e.err = SB_ERR_UNSUPPORTED;
            e.launches += 2;
        }
        if (!tiled && rem > 0) {
            AttnArgs aa{W.pf_q + (size_t)n_full * kMaxW * D.qd, k_cache_l, v_cache_l, W.page_table,
                        W.pf_attn_part + (size_t)n_full * W.pf_attn_stride, act_of(W.pf_act_o, n_full, D.qd), D.H, D.Hkv, D.hd,
                        D.page, D.page_shift, pos0 + n_full * kMaxW, 0, rem, D.chunk, nullptr, 0, W.rope_tab, W.status, {}};
            aa.pos_pred0 = pos0;   // the pass's RoPE/append launch wrote the rows of the full blocks too
            if (!launch_attention<T>(e.st, aa)) e.err = SB_ERR_UNSUPPORTED;
            e.launches += 2;
        }
    }
    const void* wo[1] = {lw.wo};
    int no[1] = {D.d};
    const int s_o = gemm(e, wo, no, 1, D.qd, W.pf_act_o, W.pf_p_o, 0, M, nullptr, NextGemm(), kWideBlocks);
    launch_resid_norm<T>(e.st, W.pf_h, W.pf_p_o, s_o, D.d, (const T*)lw.mlp_norm, D.eps, W.pf_act_a, 0, M);   // all rows
    e.launches++;
    const void* wgu[2] = {lw.w_gate, lw.w_up};
    int ngu[2] = {D.F, D.F};
    gemm(e, wgu, ngu, 2, D.d, W.pf_act_a, nullptr, 0, M, W.pf_act_f, NextGemm(), kWideBlocks);   // SwiGLU in the epilogue
    const void* wd[1] = {lw.w_down};
    int nd[1] = {D.d};
    const int s_d = gemm(e, wd, nd, 1, D.F, W.pf_act_f, W.pf_p_down, 0, M, nullptr, NextGemm(), kWideBlocks);
    launch_resid_norm<T>(e.st, W.pf_h, W.pf_p_down, s_d, D.d, (const T*)next_gain, D.eps, W.pf_act_a, 0, M);
    e.launches++;
}

// exit-confidence / final-head kernel on rows r0 .. r0+m-1; act_a must hold their final RMSNorm
static void head(Exec& e, const void* lm_head, int r0, int m, float tau, float threshold, float* conf, int* token,
                 int* flag, float* logits_dbg, const Mirror& mirror = Mirror{nullptr, nullptr, 0u}) {
    HeadArgs a{lm_head, e.D.V, e.D.d, e.W.act_a, r0, m, 1.f / tau, threshold, conf, token, flag, logits_dbg,
               e.W.head_part, e.W.ticket, mirror};
    e.launches++;
    if (e.gemm == 1 && !e.D.f32) {
        if (!launch_head_tc(e.st, a, e.plans, e.W.status)) e.err = SB_ERR_CUDA;
        return;
    }
    SB_T(e, launch_head_simt<T>(e.st, a, 148 * 4));
}

}  // namespace sb

using namespace sb;

struct sb_ctx {
    sb_config cfg;
    Exec e;
    sb_weights w;
    sb_layer_weights layers[SB_MAX_LAYERS];
    const void* exit_head[SB_MAX_LAYERS];   // per-layer exit heads / norm gains, null = shared (copied from sb_weights)
    const void* exit_norm[SB_MAX_LAYERS];
    const void* head_of(int layer) const { return exit_head[layer - 1] ? exit_head[layer - 1] : w.lm_head; }
    const void* norm_of(int layer) const { return exit_norm[layer - 1] ? exit_norm[layer - 1] : w.final_norm; }
    bool loaded = false;
    int* mailbox = nullptr;      // pinned host memory, mapped into the device's address space
    int* mailbox_dev = nullptr;  // its device address (null: the device cannot map host memory; results are copied)
    unsigned int seq = 0;        // sequence number of the last mirrored result block
    struct { int layer = 0, r0 = 0, m = 0, s_qkv = 0; } ahead;   // QKV issued ahead for the next layer step (layer 0: none)
    int64_t probes_at[SB_MAX_LAYERS + 1] = {}, exits_at[SB_MAX_LAYERS + 1] = {};   // per layer, of the current sb_generate call
    int64_t probes_issued = 0;
    bool time_round = true;      // the current round of sb_generate is bracketed by events (one round in kTimedRoundEvery)
    bool round_ahead = false;    // sb_generate: verify_rows may issue the start of the next round behind the acceptance kernel
    bool embed_ahead = false;    // ... and did: row 0 already holds the embedding of the last emitted token
    int n = 0, pending = -1, rows = 0;
    int depth[SB_MAX_W];
    float sample_temperature = 0.f;      // sampling decoding (Section 4.3): 0 = greedy
    float sample_top_p = 1.f;            // nucleus mass; 1 = the whole vocabulary
    unsigned long long sample_seed = 0;
    cudaEvent_t ev[9];   // 0 draft start, 1 verify start, 2 round end, 3/4 unified pass, 5/6 probe kernel, 7/8 decode phase
    int64_t h2d = 0, d2h = 0;
    TcPlanCache plans;

    void* kc(int layer) const {
        size_t es = e.D.f32 ? 4 : 2;
        return (char*)e.W.k_cache + es * (size_t)(layer - 1) * e.D.n_pages * e.D.page * e.D.kvd;
    }
    void* vc(int layer) const {
        size_t es = e.D.f32 ? 4 : 2;
        return (char*)e.W.v_cache + es * (size_t)(layer - 1) * e.D.n_pages * e.D.page * e.D.kvd;
    }
    float* conf_d() const { return reinterpret_cast<float*>(e.W.res); }
    int* token_d() const { return e.W.res + 8; }
    int* flag_d() const { return e.W.res + 16; }
    int* accept_d() const { return e.W.res + 24; }
};

static double now_us() {
    return std::chrono::duration<double, std::micro>(std::chrono::steady_clock::now().time_since_epoch()).count();
}

static int cuda_ok(cudaError_t err) { return err == cudaSuccess ? SB_OK : SB_ERR_CUDA; }

// copy the result block (40 words + the status word at 48) to the pinned mailbox and wait for it; also surfaces launch errors
// and expired device waits
static int fetch_results(sb_ctx* c) {
    if (cudaMemcpyAsync(c->mailbox, c->e.W.res, sizeof(int) * 49, cudaMemcpyDeviceToHost, c->e.st) != cudaSuccess)
        return SB_ERR_CUDA;
    if (report_cuda("stream synchronize", cudaStreamSynchronize(c->e.st)) != cudaSuccess) return SB_ERR_CUDA;
    if (report_cuda("last error", cudaGetLastError()) != cudaSuccess) return SB_ERR_CUDA;
    if (c->e.err) return c->e.err;
    c->d2h += sizeof(int) * 49;
    if (c->mailbox[48] != 0) return SB_ERR_DEVICE_TIMEOUT;
    return SB_OK;
}

// The kernel launched last mirrors the result block into the mailbox (publish_results) and then writes c->seq into
// word 63: poll that word instead of copying and synchronising.  Falls back to the copy if nothing arrives in time
// (a launch that failed never writes; the synchronisation then reports why).
static Mirror next_mirror(sb_ctx* c) {
    if (!c->mailbox_dev) return Mirror{nullptr, nullptr, 0u};
    return Mirror{c->mailbox_dev, c->e.W.res, ++c->seq};
}
static int wait_results(sb_ctx* c, const Mirror& m) {
    if (!m.host) return fetch_results(c);
    volatile unsigned int* flag = reinterpret_cast<volatile unsigned int*>(c->mailbox) + 63;
    const double t0 = now_us();
    for (unsigned int spins = 1; *flag != m.seq; ++spins)
        if ((spins & 4095u) == 0 && now_us() - t0 > 2e6) return fetch_results(c);
    __atomic_thread_fence(__ATOMIC_ACQUIRE);
    if (c->e.err) return c->e.err;
    c->d2h += sizeof(int) * 50;
    if (c->mailbox[48] != 0) return SB_ERR_DEVICE_TIMEOUT;
    return SB_OK;
}

static void run_layer(sb_ctx* c, int layer, int r0, int m, const void* next_gain, const void* next_gain2 = nullptr) {
    // a QKV issued ahead is good for the very next layer step only (the scratch it wrote is reused by every step)
    const int s_ahead = (c->ahead.layer == layer && c->ahead.r0 == r0 && c->ahead.m == m) ? c->ahead.s_qkv : 0;
    c->ahead.layer = 0;
    layer_step(c->e, c->layers[layer - 1], c->kc(layer), c->vc(layer), r0, m, c->n, next_gain, s_ahead, next_gain2);
    for (int i = r0; i < r0 + m; ++i) c->depth[i] = layer;
}

// run layer `layer` on the trailing rows whose depth is layer-1; returns rows advanced
// The decoding rule at the last layer for rows [r0, r0+m) (their final-norm activation is in place): greedy top-1
// from the fused head kernel, or, under sampling decoding (Section 4.3), the head kernel writes the logits and the
// sampling kernel draws token[r0 + j] at the uniform number of sequence position pos0 + j.  `mir` is published by
// whichever kernel runs last.
static void final_tokens(sb_ctx* c, int r0, int m, long long pos0, int* token, const Mirror& mir) {
    Exec& e = c->e;
    if (c->sample_temperature <= 0.f) {
        head(e, c->w.lm_head, r0, m, 1.f, 2.f, c->conf_d(), token, c->flag_d(), nullptr, mir);
        return;
    }
    head(e, c->w.lm_head, r0, m, 1.f, 2.f, c->conf_d(), c->token_d(), c->flag_d(), e.W.logits);
    SampleArgs a{e.W.logits, e.W.sample_e, e.W.sample_q, e.D.V, r0, m, (double)c->sample_temperature, (double)c->sample_top_p, c->sample_seed, pos0, token,
                 reinterpret_cast<unsigned int*>(e.W.res + 57), mir};
    if (!launch_sample(e.st, a)) e.err = SB_ERR_CUDA;
    e.launches++;
}

static int advance_suffix(sb_ctx* c, int layer, const void* next_gain, sb_stats* st, const void* next_gain2 = nullptr) {
    int r0 = c->rows;
    while (r0 > 0 && c->depth[r0 - 1] == layer - 1) --r0;
    int m = c->rows - r0;
    if (m == 0) return 0;
    run_layer(c, layer, r0, m, next_gain, next_gain2);
    if (st) { st->layer_steps++; st->layer_row_steps += m; }
    return m;
}

// ---------------------------------------------------------------------------------------------
// Scratch of sb_k_exit_confidence_static: a fixed array in device memory that exists as soon as the
// library is loaded on a GPU, so the call needs no allocation from anybody.  Shared by all calls.
// ---------------------------------------------------------------------------------------------
constexpr size_t kStaticScratchBytes = size_t(1) << 20;   // 1 MiB
constexpr int kStaticMaxDModel = 8192;                    // widest model whose rows fit it
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// what the exit-confidence call keeps in scratch: hidden rows, the normalised operand, the per-CTA
// softmax triples, the ticket, the result block and the status word
static size_t carve_exit_only(const Dims& D, char* base, Work* w) {
    Carver c{base};
    Work tmp;
    Work& W = w ? *w : tmp;
    size_t es = D.f32 ? 4 : 2, act_rows = D.f32 ? 8 : 16;
    c.take(W.h, sizeof(float) * kMaxW * D.d);
    c.take(W.act_a, es * act_rows * D.d);
    c.take(W.head_part, sizeof(SoftTriple) * kHeadMaxCtas * kMaxW);
    c.take(W.res, sizeof(int) * 64);
    W.status = reinterpret_cast<unsigned int*>(W.res + 48);   // status word and ticket inside the result block, as in carve()
    W.ticket = reinterpret_cast<unsigned int*>(W.res + 56);
    return (c.off + 1023) & ~size_t(1023);
}

// Device address of the static scratch on the current device.  In host code the array's name is
// only a host-side handle, never a device address: the address comes from cudaGetSymbolAddress,
// asked once per device with that device current.
static int static_scratch_ptr(char** out) {
    static char* ptrs[kMaxDevices] = {nullptr};
    const int dev = current_device();
    if (dev < 0) return SB_ERR_CUDA;
    if (!ptrs[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) {
            (void)cudaGetLastError();
            return SB_ERR_CUDA;
        }
        ptrs[dev] = static_cast<char*>(p);
    }
    *out = ptrs[dev];
    return SB_OK;
}

extern "C" {

size_t sb_workspace_bytes(const sb_config* cfg) {
    Dims D;
    if (!make_dims(cfg, &D)) return 0;
    return carve(D, nullptr, true, nullptr);
}

size_t sb_k_scratch_bytes(const sb_config* cfg) {
    Dims D;
    if (!make_dims(cfg, &D)) return 0;
    return carve(D, nullptr, false, nullptr);
}

int sb_create(const sb_config* cfg, void* workspace, size_t bytes, void* stream, sb_ctx** out) {
    Dims D;
    if (!out || !workspace || !make_dims(cfg, &D)) return SB_ERR_ARG;
    if ((uintptr_t)workspace & 1023) return SB_ERR_ARG;
    if (bytes < carve(D, nullptr, true, nullptr)) return SB_ERR_CAPACITY;
    sb_ctx* c = new (std::nothrow) sb_ctx();
    if (!c) return SB_ERR_CUDA;
    c->cfg = *cfg;
    c->e.D = D;
    c->e.st = (cudaStream_t)stream;
    carve(D, (char*)workspace, true, &c->e.W);
    c->e.gemm = pick_gemm(D.f32);
    c->e.plans = &c->plans;
    if (cudaHostAlloc((void**)&c->mailbox, sizeof(int) * 64, cudaHostAllocMapped) != cudaSuccess) {
        delete c;
        return SB_ERR_CUDA;
    }
    memset(c->mailbox, 0, sizeof(int) * 64);
    if (cudaHostGetDevicePointer((void**)&c->mailbox_dev, c->mailbox, 0) != cudaSuccess) {
        (void)cudaGetLastError();
        c->mailbox_dev = nullptr;
    }
    for (auto& ev : c->ev) cudaEventCreate(&ev);
    launch_init_pages(c->e.st, c->e.W.page_table, D.n_pages);
    launch_rope_table(c->e.st, c->e.W.rope_tab, D.n_pages * D.page, D.hd / 2, D.inv_freq);
    cudaMemsetAsync(c->e.W.res, 0, sizeof(int) * 64, c->e.st);   // results, status word (48) and ticket (56)
    if (cudaStreamSynchronize(c->e.st) != cudaSuccess || cudaGetLastError() != cudaSuccess) {
        sb_destroy(c);
        return SB_ERR_CUDA;
    }
    for (int i = 0; i < SB_MAX_W; ++i) c->depth[i] = 0;
    *out = c;
    return SB_OK;
}

void sb_destroy(sb_ctx* c) {
    if (!c) return;
    cudaStreamSynchronize(c->e.st);
    for (auto& ev : c->ev) cudaEventDestroy(ev);
    if (c->mailbox) cudaFreeHost(c->mailbox);
    delete c;
}

int sb_load_weights(sb_ctx* c, const sb_weights* w) {
    if (!c || !w || !w->embed || !w->final_norm || !w->lm_head || !w->layers) return SB_ERR_ARG;
    auto bad = [](const void* p) { return !p || ((uintptr_t)p & 15); };
    if (bad(w->embed) || bad(w->final_norm) || bad(w->lm_head)) return SB_ERR_ARG;
    for (int l = 0; l < c->e.D.L; ++l) {
        const sb_layer_weights& s = w->layers[l];
        const void* ps[9] = {s.attn_norm, s.wq, s.wk, s.wv, s.wo, s.mlp_norm, s.w_gate, s.w_up, s.w_down};
        for (const void* p : ps)
            if (bad(p)) return SB_ERR_ARG;
    }
    for (int l = 0; l < c->e.D.L; ++l) {
        const void* eh = w->exit_head ? w->exit_head[l] : nullptr;
        const void* en = w->exit_norm ? w->exit_norm[l] : nullptr;
        if (((uintptr_t)eh & 15) || ((uintptr_t)en & 15)) return SB_ERR_ARG;
    }
    c->w = *w;
    for (int l = 0; l < c->e.D.L; ++l) {
        c->layers[l] = w->layers[l];
        c->exit_head[l] = w->exit_head ? w->exit_head[l] : nullptr;
        c->exit_norm[l] = w->exit_norm ? w->exit_norm[l] : nullptr;
    }
    c->w.layers = c->layers;
    c->w.exit_head = c->exit_head;
    c->w.exit_norm = c->exit_norm;
    c->plans.clear();
    c->loaded = true;
    return SB_OK;
}

int sb_reset(sb_ctx* c) {
    if (!c) return SB_ERR_ARG;
    c->n = 0; c->pending = -1; c->rows = 0;
    c->ahead.layer = 0; c->embed_ahead = false; c->round_ahead = false;
    c->e.act_gain = nullptr; c->e.act2_gain = nullptr;
    // a sticky host error or an expired device wait of an earlier call is forgotten with the sequence
    c->e.err = 0;
    if (cudaMemsetAsync(c->e.W.status, 0, 64, c->e.st) != cudaSuccess) return SB_ERR_CUDA;
    return SB_OK;
}

int sb_selftest_wait_timeout(sb_ctx* c, int32_t budget_ms) {
    if (!c || budget_ms < 1 || budget_ms > 1000) return SB_ERR_ARG;
    // the kernel reports through the context's own status word and the last word of the result block
    unsigned int* flag = reinterpret_cast<unsigned int*>(c->e.W.res) + 63;
    cudaMemsetAsync(flag, 0, sizeof(unsigned int), c->e.st);
    launch_wait_selftest(c->e.st, c->e.W.status, (unsigned long long)budget_ms * 2000000ull, flag);
    int rc = fetch_results(c);   // SB_ERR_DEVICE_TIMEOUT when the wait gave up, as it must
    unsigned int f = 0;
    if (cudaMemcpy(&f, flag, sizeof(f), cudaMemcpyDeviceToHost) != cudaSuccess) return SB_ERR_CUDA;
    if (rc == SB_ERR_DEVICE_TIMEOUT && f != 2u) return SB_ERR_STATE;
    return rc;
}

int sb_get_state(sb_ctx* c, sb_state* out) {
    if (!c || !out) return SB_ERR_ARG;
    out->n = c->n; out->pending = c->pending; out->rows = c->rows;
    for (int i = 0; i < SB_MAX_W; ++i) out->depth[i] = i < c->rows ? c->depth[i] : 0;
    return SB_OK;
}

int sb_read_hidden(sb_ctx* c, int32_t row, float* host_out) {
    if (!c || !host_out || row < 0 || row >= c->rows) return SB_ERR_ARG;
    if (cudaMemcpyAsync(host_out, c->e.W.h + (size_t)row * c->e.D.d, sizeof(float) * c->e.D.d, cudaMemcpyDeviceToHost,
                        c->e.st) != cudaSuccess)
        return SB_ERR_CUDA;
    return cuda_ok(cudaStreamSynchronize(c->e.st));
}

int sb_set_option(sb_ctx* c, int32_t key, int32_t value) {
    if (!c) return SB_ERR_ARG;
    if (key == SB_OPT_GEMM) {
        if (value != 0 && value != 1) return SB_ERR_ARG;
        if (value == 1 && (c->e.D.f32 || !tc_available())) return SB_ERR_UNSUPPORTED;
        c->e.gemm = value;
        return SB_OK;
    }
    return SB_ERR_ARG;
}

int sb_set_default_option(int32_t key, int32_t value) {
    if (key == SB_OPT_TRACE) { g_trace = value != 0; return SB_OK; }
    if (key == SB_OPT_L2_PREFETCH) return tc_set_l2_prefetch(value) ? SB_OK : SB_ERR_ARG;
    if (key == SB_OPT_SPLIT_PENALTY) return tc_set_split_penalty(value) ? SB_OK : SB_ERR_ARG;
    if (key == SB_OPT_QKV_AHEAD) { g_qkv_ahead = value != 0; return SB_OK; }
    if (key == SB_OPT_WIDE_PREFILL) {
        if (value < 0 || value > 3) return SB_ERR_ARG;
        g_wide_prefill = value;
        tc_set_wide_cta_pairs(value != 3);
        return SB_OK;
    }
    if (key == SB_OPT_PDL) { g_use_pdl = value != 0; return SB_OK; }
    if (key == SB_OPT_FUSE) { if (value < 0 || value > 3) return SB_ERR_ARG; g_fuse = value; return SB_OK; }
    if (key == SB_OPT_TC_TUNING) return tc_set_tuning(value / 16, value % 16) ? SB_OK : SB_ERR_ARG;
    if (key == SB_OPT_GEMM && (value == 0 || value == 1 || value == -1)) {
        if (value == 1 && !tc_available()) return SB_ERR_UNSUPPORTED;
        g_default_gemm = value;
        return SB_OK;
    }
    return SB_ERR_ARG;
}

int sb_set_sampling(sb_ctx* c, float temperature, float top_p, uint64_t seed) {
    if (!c || temperature != temperature || temperature < 0.f || !(top_p > 0.f) || top_p > 1.f) return SB_ERR_ARG;
    if (temperature > 0.f && c->e.D.V > kSampleMaxVocab) return SB_ERR_CAPACITY;
    c->sample_temperature = temperature;
    c->sample_top_p = top_p;
    c->sample_seed = seed;
    return SB_OK;
}

double sb_sample_uniform(uint64_t seed, int64_t pos) { return sample_uniform(seed, pos); }

static int check_tokens(const sb_ctx* c, const int32_t* t, int n) {
    for (int i = 0; i < n; ++i)
        if (t[i] < 0 || t[i] >= c->e.D.V) return SB_ERR_ARG;
    return SB_OK;
}

int sb_prefill(sb_ctx* c, const int32_t* prompt, int32_t n_prompt, int32_t* first_token) {
    if (!c || !prompt || !first_token || n_prompt < 1) return SB_ERR_ARG;
    if (!c->loaded) return SB_ERR_STATE;
    if (c->n != 0 || c->rows != 0) return SB_ERR_STATE;
    if (n_prompt + 1 > c->e.D.max_seq) return SB_ERR_CAPACITY;
    if (check_tokens(c, prompt, n_prompt)) return SB_ERR_ARG;
    Exec& e = c->e;
    if (cudaMemcpyAsync(e.W.toks, prompt, sizeof(int) * n_prompt, cudaMemcpyHostToDevice, e.st) != cudaSuccess)
        return SB_ERR_CUDA;
    c->h2d += sizeof(int) * n_prompt;
    int m = 0;
    int done = 0;
    // Wide passes (bf16 models on the tcgen05 path with the SwiGLU epilogue): up to 128 prompt rows per pass, so the
    // weights are streamed once per 128 rows; what is left over (fewer than 16 rows) goes through 8-row passes below.
    if (tc_path(e) && (g_fuse & 1) && g_wide_prefill && e.W.pf_h) {
        while (n_prompt - done >= 2 * kMaxW) {
            const int M = n_prompt - done < kWideRows ? n_prompt - done : kWideRows;
            launch_embed<__nv_bfloat16>(e.st, (const __nv_bfloat16*)c->w.embed, e.D.d, e.W.toks + done, 0, 0, M, e.W.pf_h);
            e.launches++;
            for (int l = 1; l <= e.D.L; ++l)
                layer_step_wide(e, c->layers[l - 1], c->kc(l), c->vc(l), M, done, l > 1,
                                l < e.D.L ? c->layers[l].attn_norm : nullptr);
            done += M;
            if (done == n_prompt) {   // the last 8-row block's hidden rows are what the first generated token comes from
                const int nblk = (M + kMaxW - 1) / kMaxW;
                m = M - (nblk - 1) * kMaxW;
                if (cudaMemcpyAsync(e.W.h, e.W.pf_h + (size_t)(nblk - 1) * kMaxW * e.D.d, sizeof(float) * m * e.D.d,
                                    cudaMemcpyDeviceToDevice, e.st) != cudaSuccess)
                    return SB_ERR_CUDA;
                e.act_gain = nullptr; e.act2_gain = nullptr;
            }
        }
    }
    for (int p0 = done; p0 < n_prompt; p0 += m) {
        m = n_prompt - p0 < kMaxW ? n_prompt - p0 : kMaxW;
        bool last = p0 + m == n_prompt;
        SB_T(e, launch_embed<T>(e.st, (const T*)c->w.embed, e.D.d, e.W.toks + p0, 0, 0, m, e.W.h));
        e.launches++;
        e.act_gain = nullptr; e.act2_gain = nullptr;
        c->n = p0;
        for (int l = 1; l <= e.D.L; ++l) {
            const void* next = l < e.D.L ? c->layers[l].attn_norm : (last ? c->w.final_norm : nullptr);
            layer_step(e, c->layers[l - 1], c->kc(l), c->vc(l), 0, m, c->n, next);
        }
    }
    c->n = n_prompt;
    ensure_act(e, c->w.final_norm, m - 1, 1);
    const Mirror mir = next_mirror(c);
    final_tokens(c, m - 1, 1, n_prompt, c->token_d(), mir);
    int rc = wait_results(c, mir);
    if (rc) return rc;
    c->pending = c->mailbox[8 + (m - 1)];
    c->rows = 0;
    *first_token = c->pending;
    return SB_OK;
}

// from_generate: the call comes from sb_generate's round loop, which alone may have issued the embedding ahead
static int draft_push(sb_ctx* c, int32_t token, bool from_generate) {
    if (!c) return SB_ERR_ARG;
    if (!from_generate) c->embed_ahead = false;
    if (!c->loaded || c->pending < 0) return SB_ERR_STATE;
    if (token < 0 || token >= c->e.D.V) return SB_ERR_ARG;
    if (c->rows >= SB_MAX_W) return SB_ERR_CAPACITY;
    if (c->n + c->rows + 1 > c->e.D.max_seq) return SB_ERR_CAPACITY;
    Exec& e = c->e;
    if (c->embed_ahead && c->rows == 0) {
        c->embed_ahead = false;   // issued behind the last round's acceptance kernel, from the same token on the device
    } else {
        SB_T(e, launch_embed<T>(e.st, (const T*)c->w.embed, e.D.d, nullptr, token, c->rows, 1, e.W.h));
        e.launches++;
    }
    c->depth[c->rows++] = 0;
    return SB_OK;
}
int sb_draft_push(sb_ctx* c, int32_t token) { return draft_push(c, token, false); }

int sb_draft_advance(sb_ctx* c, int32_t to_layer) {
    if (!c) return SB_ERR_ARG;
    if (!c->loaded || c->rows < 1) return SB_ERR_STATE;
    if (to_layer < 1 || to_layer > c->e.D.L) return SB_ERR_ARG;
    for (int l = 1; l <= to_layer; ++l) advance_suffix(c, l, c->norm_of(l), nullptr);
    return cuda_ok(cudaGetLastError());
}

// While the host waits for the exit decision after layer `layer`, the GPU would idle: issue the norm + QKV GEMM of
// the layer step that follows if the row does not exit (rows of the trailing run at depth `layer`).  If it exits,
// the work is discarded: nothing but scratch was written.
static void qkv_ahead(sb_ctx* c, int layer) {
    if (!g_qkv_ahead || layer >= c->e.D.L) return;
    // not where rows usually exit (the work would be thrown away more often than used)
    if (c->probes_at[layer] >= 8 && 3 * c->exits_at[layer] > c->probes_at[layer]) return;
    int r0 = c->rows;
    while (r0 > 0 && c->depth[r0 - 1] == layer) --r0;
    const int m = c->rows - r0;
    if (m < 1) return;
    c->ahead.s_qkv = layer_qkv(c->e, c->layers[layer], r0, m);   // layers[layer] = layer number layer + 1
    c->ahead.layer = layer + 1; c->ahead.r0 = r0; c->ahead.m = m;
}

// sb_generate brackets one round in this many with CUDA events (phase times, the unified pass's time and counters)
constexpr int kTimedRoundEvery = 4;

static int probe(sb_ctx* c, int layer, float tau_l, float threshold, float* conf, int32_t* token, int32_t* flag,
                 sb_stats* st = nullptr, bool more_layers = false) {
    int r = c->rows - 1;
    ensure_act(c->e, c->norm_of(layer), r, 1);
    // One probe in 32 is bracketed by events (which needs the copy + synchronise path and keeps the kernel from
    // overlapping its predecessor); the others report through the mirror.
    const bool timed = st && (c->probes_issued++ & 31) == 0;
    if (timed) {
        cudaEventRecord(c->ev[5], c->e.st);
        head(c->e, c->head_of(layer), r, 1, tau_l, threshold, c->conf_d(), c->token_d(), c->flag_d(), nullptr);
        cudaEventRecord(c->ev[6], c->e.st);
        if (more_layers) qkv_ahead(c, layer);
        int rc = fetch_results(c);
        if (rc) return rc;
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, c->ev[5], c->ev[6]) == cudaSuccess) { st->us_probe_kernels += 1e3 * ms; st->probes_timed++; }
    } else {
        const Mirror mir = next_mirror(c);
        head(c->e, c->head_of(layer), r, 1, tau_l, threshold, c->conf_d(), c->token_d(), c->flag_d(), nullptr, mir);
        if (more_layers) qkv_ahead(c, layer);
        int rc = wait_results(c, mir);
        if (rc) return rc;
    }
    memcpy(conf, &c->mailbox[r], sizeof(float));
    *token = c->mailbox[8 + r];
    *flag = c->mailbox[16 + r];
    (void)layer;
    return SB_OK;
}

int sb_exit_confidence(sb_ctx* c, int32_t layer, float tau_l, float threshold, float* conf, int32_t* token,
                       int32_t* exit_flag) {
    if (!c || !conf || !token || !exit_flag) return SB_ERR_ARG;
    if (!c->loaded || c->rows < 1) return SB_ERR_STATE;
    if (layer < 1 || layer > c->e.D.L || !(tau_l > 0.f) || threshold != threshold) return SB_ERR_ARG;
    if (c->depth[c->rows - 1] != layer) return SB_ERR_STATE;
    return probe(c, layer, tau_l, threshold, conf, token, exit_flag);
}

// alignment + unified pass + final head + acceptance + rollback
static int verify_rows(sb_ctx* c, const int32_t* drafts, int w, int max_emit, int32_t* out_tokens, int32_t* n_out,
                       sb_stats* st, sb_round* tr) {
    Exec& e = c->e;
    int D = 0;
    for (int i = 0; i < w; ++i) D = c->depth[i] > D ? c->depth[i] : D;
    for (int l = 1; l <= D; ++l) advance_suffix(c, l, l < e.D.L ? c->layers[l].attn_norm : c->w.final_norm, st);
    c->ahead.layer = 0;   // the unified pass is timed as a whole: it never starts from work issued ahead of its window
    // An event between two kernels keeps the second from overlapping the first (its weight tiles are requested only
    // after the event): the rounds that are timed pay a few microseconds per event, so only some are (sb_generate).
    const bool timed = st && c->time_round;
    if (timed) cudaEventRecord(c->ev[3], e.st);
    for (int l = D + 1; l <= e.D.L; ++l) {
        run_layer(c, l, 0, w, l < e.D.L ? c->layers[l].attn_norm : c->w.final_norm);
        if (st) { st->layer_steps++; st->layer_row_steps += w; }
        if (timed) { st->unified_layer_steps++; st->unified_kv_positions += c->n + w; }
    }
    if (timed) cudaEventRecord(c->ev[4], e.st);
    ensure_act(e, c->w.final_norm, 0, w);
    final_tokens(c, 0, w, (long long)c->n + 1, c->token_d(), Mirror{nullptr, nullptr, 0u});   // row i holds position n + i
    int d8[kMaxW];
    for (int i = 0; i < kMaxW; ++i) d8[i] = i < w ? drafts[i] : -1;
    const Mirror mir = next_mirror(c);
    launch_accept(e.st, c->token_d(), d8, w, max_emit, c->accept_d(), mir);
    e.launches++;
    if (timed) cudaEventRecord(c->ev[2], e.st);
    // While the host waits for the outcome, the GPU would idle: the next round always starts by embedding the last
    // emitted token, which the acceptance kernel has left on the device, and by the RMSNorm + QKV GEMM of layer 1 on
    // row 0.  They touch the hidden row, the operand buffer and scratch only (the rows of this round are done with).
    if (c->round_ahead && e.D.L > 1) {
        SB_T(e, launch_embed<T>(e.st, (const T*)c->w.embed, e.D.d, c->accept_d() + 10, 0, 0, 1, e.W.h));
        e.launches++;
        e.act_gain = nullptr; e.act2_gain = nullptr;
        c->ahead.s_qkv = layer_qkv(e, c->layers[0], 0, 1);
        c->ahead.layer = 1; c->ahead.r0 = 0; c->ahead.m = 1;
        c->embed_ahead = true;
    }
    int rc = wait_results(c, mir);
    if (rc) return rc;
    if (timed) cudaEventSynchronize(c->ev[2]);   // the round's events are read below and by the caller
    if (timed) {
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, c->ev[3], c->ev[4]) == cudaSuccess) st->us_unified += 1e3 * ms;
    }
    int emit = c->mailbox[24], acc = c->mailbox[25];
    for (int i = 0; i < emit; ++i) out_tokens[i] = c->mailbox[26 + i];
    *n_out = emit;
    if (tr) {
        tr->w = w; tr->D = D; tr->emitted = emit; tr->accepted_drafts = acc;
        for (int i = 0; i < kMaxW; ++i) { tr->g[i] = c->mailbox[26 + i]; tr->draft[i] = d8[i]; }
    }
    if (st) { st->accepted_drafts += acc; st->emitted += emit; st->rounds++; st->rows += w; st->width_hist[w]++; }
    c->n += emit;                       // rollback: KV at positions >= n is dead and will be overwritten
    c->pending = c->mailbox[26 + emit - 1];
    c->rows = 0;
    e.act_gain = nullptr; e.act2_gain = nullptr;
    return SB_OK;
}

int sb_verify(sb_ctx* c, const int32_t* drafts, int32_t w, int32_t* out_tokens, int32_t* n_out) {
    if (!c || !drafts || !out_tokens || !n_out) return SB_ERR_ARG;
    if (!c->loaded) return SB_ERR_STATE;
    if (w < 1 || w > SB_MAX_W) return SB_ERR_ARG;
    if (w != c->rows) return SB_ERR_STATE;
    for (int i = 0; i < w; ++i)
        if (drafts[i] < -1 || drafts[i] >= c->e.D.V) return SB_ERR_ARG;
    return verify_rows(c, drafts, w, w, out_tokens, n_out, nullptr, nullptr);
}


int sb_generate(sb_ctx* c, const int32_t* prompt, int32_t n_prompt, int32_t n_gen, int32_t d_max, int32_t w_max,
                const float* tau, float threshold, int32_t* out_tokens, int32_t* n_out, sb_stats* stats,
                sb_round* rounds, int32_t max_rounds, int32_t* n_rounds) {
    if (!c || !prompt || !tau || !out_tokens || !n_out || n_prompt < 1 || n_gen < 1) return SB_ERR_ARG;
    if (!c->loaded) return SB_ERR_STATE;
    if (d_max < 1 || d_max > c->e.D.L - 1 || w_max < 1 || w_max > SB_MAX_W || threshold != threshold) return SB_ERR_ARG;
    for (int l = 0; l < d_max; ++l)
        if (tau[l] != tau[l]) return SB_ERR_ARG;   // NaN; tau[l] <= 0 = layer l + 1 is not probed
    if (n_prompt + n_gen + w_max > c->e.D.max_seq) return SB_ERR_CAPACITY;
    if (check_tokens(c, prompt, n_prompt)) return SB_ERR_ARG;
    sb_stats local;
    sb_stats* st = stats ? stats : &local;
    memset(st, 0, sizeof(*st));
    memset(c->probes_at, 0, sizeof(c->probes_at));
    memset(c->exits_at, 0, sizeof(c->exits_at));
    Exec& e = c->e;
    int64_t launches0 = e.launches, h2d0 = c->h2d, d2h0 = c->d2h;
    sb_reset(c);
    double t0 = now_us();
    int first;
    int rc = sb_prefill(c, prompt, n_prompt, &first);
    if (rc) return rc;
    double t1 = now_us();
    st->us_prefill = t1 - t0;
    cudaEventRecord(c->ev[7], e.st);
    int produced = 0, nr = 0;
    out_tokens[produced++] = first;
    st->emitted = 1;
    while (produced < n_gen) {
        sb_round R;
        memset(&R, 0, sizeof(R));
        int drafts[kMaxW];
        for (int i = 0; i < kMaxW; ++i) { drafts[i] = -1; R.draft[i] = -1; }
        int cur = c->pending;
        c->time_round = (nr % kTimedRoundEvery) == 0;
        if (c->time_round) cudaEventRecord(c->ev[0], e.st);
        for (;;) {                              // draft phase (Section 3.3)
            if ((rc = draft_push(c, cur, true))) return rc;
            int r = c->rows - 1;
            bool exited = false;
            for (int l = 1; l <= d_max; ++l) {
                // a layer whose temperature is <= 0 is walked but not probed: its step hands the rows straight to the
                // next layer's attention norm
                const bool probed = tau[l - 1] > 0.f;
                // a probed layer leaves its rows under the exit test's norm and, for the step that follows if the row
                // stays, under the next layer's attention norm as well (one RMSNorm launch less per exit test)
                advance_suffix(c, l, probed ? c->norm_of(l) : c->layers[l].attn_norm, st,
                               probed && l < e.D.L ? c->layers[l].attn_norm : nullptr);
                if (!probed) continue;
                float conf; int tok, flag;
                if ((rc = probe(c, l, tau[l - 1], threshold, &conf, &tok, &flag, st, l < d_max))) return rc;
                st->probes++;
                c->probes_at[l]++;
                if (flag) c->exits_at[l]++;
                R.conf[r] = conf;
                if (flag) { drafts[r] = tok; R.exit_layer[r] = l; exited = true; break; }
            }
            st->exit_hist[exited ? R.exit_layer[r] : 0]++;
            if (!exited) break;                 // difficult token: the depth bound ends the round
            if (c->rows == w_max) break;        // long shallow chain: the width bound ends the round
            cur = drafts[r];
        }
        if (c->time_round) cudaEventRecord(c->ev[1], e.st);
        int w = c->rows, emit = 0;
        c->round_ahead = g_qkv_ahead && produced + w < n_gen;   // this round cannot be the last one
        if ((rc = verify_rows(c, drafts, w, n_gen - produced, out_tokens + produced, &emit, st, &R))) return rc;
        produced += emit;
        if (c->time_round) {
            float ms = 0.f;
            if (cudaEventElapsedTime(&ms, c->ev[0], c->ev[1]) == cudaSuccess) st->us_draft += 1e3 * ms;
            if (cudaEventElapsedTime(&ms, c->ev[1], c->ev[2]) == cudaSuccess) st->us_verify += 1e3 * ms;
            st->rounds_timed++;
        }
        if (rounds && nr < max_rounds) rounds[nr] = R;
        ++nr;
    }
    c->round_ahead = false; c->embed_ahead = false; c->ahead.layer = 0;
    cudaEventRecord(c->ev[8], e.st);
    cudaEventSynchronize(c->ev[8]);
    st->us_decode = now_us() - t1;
    {
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, c->ev[7], c->ev[8]) == cudaSuccess) st->us_decode_dev = 1e3 * ms;
    }
    c->d2h += sizeof(int) * produced;   // the caller's token buffer is host memory written from the mailbox
    st->kernel_launches = e.launches - launches0;
    st->h2d_bytes = c->h2d - h2d0;
    st->d2h_bytes = c->d2h - d2h0;
    *n_out = produced;
    if (n_rounds) *n_rounds = nr;
    return SB_OK;
}

int sb_generate_ar(sb_ctx* c, const int32_t* prompt, int32_t n_prompt, int32_t n_gen, int32_t* out_tokens, int32_t* n_out,
                   sb_stats* stats) {
    if (!c || !prompt || !out_tokens || !n_out || n_prompt < 1 || n_gen < 1) return SB_ERR_ARG;
    if (!c->loaded) return SB_ERR_STATE;
    if (n_prompt + n_gen > c->e.D.max_seq) return SB_ERR_CAPACITY;
    if (check_tokens(c, prompt, n_prompt)) return SB_ERR_ARG;
    sb_stats local;
    sb_stats* st = stats ? stats : &local;
    memset(st, 0, sizeof(*st));
    Exec& e = c->e;
    int64_t launches0 = e.launches, h2d0 = c->h2d, d2h0 = c->d2h;
    sb_reset(c);
    double t0 = now_us();
    int first;
    int rc = sb_prefill(c, prompt, n_prompt, &first);
    if (rc) return rc;
    double t1 = now_us();
    st->us_prefill = t1 - t0;
    cudaEventRecord(c->ev[7], e.st);
    // token log on the device: toks[n_prompt + i] = i-th generated token.  Each step embeds the
    // previous token straight from the log, so the host never has to look at a token in between.
    int* log = e.W.toks + n_prompt;
    if (cudaMemcpyAsync(log, &first, sizeof(int), cudaMemcpyHostToDevice, e.st) != cudaSuccess) return SB_ERR_CUDA;
    for (int i = 1; i < n_gen; ++i) {
        SB_T(e, launch_embed<T>(e.st, (const T*)c->w.embed, e.D.d, log + i - 1, 0, 0, 1, e.W.h));
        e.launches++;
        e.act_gain = nullptr; e.act2_gain = nullptr;
        for (int l = 1; l <= e.D.L; ++l)
            layer_step(e, c->layers[l - 1], c->kc(l), c->vc(l), 0, 1, c->n, l < e.D.L ? c->layers[l].attn_norm : c->w.final_norm);
        final_tokens(c, 0, 1, (long long)c->n + 1, log + i, Mirror{nullptr, nullptr, 0u});
        c->n += 1;
        st->layer_steps += e.D.L; st->layer_row_steps += e.D.L; st->rounds++; st->rows++;
    }
    cudaEventRecord(c->ev[8], e.st);
    if (cudaMemcpyAsync(out_tokens, log, sizeof(int) * n_gen, cudaMemcpyDeviceToHost, e.st) != cudaSuccess)
        return SB_ERR_CUDA;
    c->d2h += sizeof(int) * n_gen;
    c->h2d += sizeof(int);
    rc = fetch_results(c);
    if (rc) return rc;
    c->pending = out_tokens[n_gen - 1];
    st->emitted = n_gen;
    st->us_decode = now_us() - t1;
    {
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, c->ev[7], c->ev[8]) == cudaSuccess) st->us_decode_dev = 1e3 * ms;
    }
    st->h2d_bytes = c->h2d - h2d0;
    st->d2h_bytes = c->d2h - d2h0;
    st->kernel_launches = e.launches - launches0;
    *n_out = n_gen;
    return SB_OK;
}

int sb_k_exit_confidence(const sb_config* cfg, const void* h, int32_t m, const void* final_norm, const void* lm_head,
                         float tau_l, float* conf, int32_t* token, float* logits_dbg, void* scratch, size_t scratch_bytes,
                         void* stream) {
    Dims D;
    if (!make_dims(cfg, &D) || !h || !final_norm || !lm_head || !conf || !token || !scratch) return SB_ERR_ARG;
    if (m < 1 || m > SB_MAX_W || !(tau_l > 0.f)) return SB_ERR_ARG;
    if (((uintptr_t)scratch & 1023) || ((uintptr_t)lm_head & 15) || ((uintptr_t)h & 15)) return SB_ERR_ARG;
    if (scratch_bytes < carve(D, nullptr, false, nullptr)) return SB_ERR_CAPACITY;
    std::lock_guard<std::mutex> lock(g_stateless_mu);
    Exec e;
    e.D = D;
    e.st = (cudaStream_t)stream;
    carve(D, (char*)scratch, false, &e.W);
    e.gemm = pick_gemm(D.f32);
    e.plans = &stateless_plans();
    // the kernels read the caller's rows and write the caller's outputs directly: the call is the RMSNorm (which also
    // clears the status word and the ticket) and the exit-confidence kernel
    e.clear_next = e.W.status;
    e.W.h = const_cast<float*>(reinterpret_cast<const float*>(h));
    ensure_act(e, final_norm, 0, m);
    head(e, lm_head, 0, m, tau_l, 2.f, conf, token, e.W.res + 16, logits_dbg);
    if (e.err) return e.err;
    return cuda_ok(cudaGetLastError());
}

// Sampling kernel alone: tokens of m rows of device logits.  Nothing is published to the host, so the kernel's
// completion counter is not used: the call touches the caller's buffers only.
size_t sb_k_sample_scratch_bytes(int32_t m, int32_t vocab) {
    return m < 1 || vocab < 1 ? 0 : 2 * sizeof(double) * (size_t)m * (size_t)vocab;   // exponentials as fp64 and as fixed point
}

int sb_k_sample(const float* logits, int32_t m, int32_t vocab, float temperature, float top_p, uint64_t seed, int64_t pos0,
                int32_t* token, void* scratch, size_t scratch_bytes, void* stream) {
    if (!logits || !token || !scratch || m < 1 || m > SB_MAX_W || vocab < 1 || !(temperature > 0.f)) return SB_ERR_ARG;
    if (((uintptr_t)scratch & 7) || scratch_bytes < sb_k_sample_scratch_bytes(m, vocab)) return SB_ERR_ARG;
    if (!(top_p > 0.f) || top_p > 1.f) return SB_ERR_ARG;
    if (vocab > kSampleMaxVocab) return SB_ERR_CAPACITY;
    SampleArgs a{logits, static_cast<double*>(scratch), static_cast<unsigned long long*>(scratch) + (size_t)m * vocab, vocab, 0, m, (double)temperature, (double)top_p, seed, pos0, token,
                 nullptr, Mirror{nullptr, nullptr, 0u}};
    if (!launch_sample((cudaStream_t)stream, a)) { (void)cudaGetLastError(); return SB_ERR_CUDA; }
    return cuda_ok(cudaGetLastError());
}

int sb_k_exit_confidence_static(const sb_config* cfg, const void* h, int32_t m, const void* final_norm,
                                const void* lm_head, float tau_l, float* conf, int32_t* token, void* stream) {
    Dims D;
    if (cfg && cfg->d_model > kStaticMaxDModel) return SB_ERR_CAPACITY;   // would not fit the fixed array
    if (!make_dims(cfg, &D) || !h || !final_norm || !lm_head || !conf || !token) return SB_ERR_ARG;
    if (m < 1 || m > SB_MAX_W || !(tau_l > 0.f)) return SB_ERR_ARG;
    if (((uintptr_t)lm_head & 15) || ((uintptr_t)h & 15)) return SB_ERR_ARG;
    if (carve_exit_only(D, nullptr, nullptr) > kStaticScratchBytes) return SB_ERR_CAPACITY;
    char* base = nullptr;
    int rc = static_scratch_ptr(&base);   // first call on a device looks the address up
    if (rc) return rc;
    std::lock_guard<std::mutex> lock(g_stateless_mu);
    Exec e;
    e.D = D;
    e.st = (cudaStream_t)stream;
    e.W = Work{};
    carve_exit_only(D, base, &e.W);
    e.gemm = pick_gemm(D.f32);
    e.plans = &stateless_plans();
    // the array keeps whatever the previous call left: the status word and the ticket must start at zero (the RMSNorm
    // launch clears them)
    e.clear_next = e.W.status;
    e.W.h = const_cast<float*>(reinterpret_cast<const float*>(h));
    ensure_act(e, final_norm, 0, m);
    head(e, lm_head, 0, m, tau_l, 2.f, conf, token, e.W.res + 16, nullptr);
    if (e.err) return e.err;
    return cuda_ok(cudaGetLastError());
}

int sb_k_layer(const sb_config* cfg, const sb_layer_weights* lw, void* h, int32_t m, void* k_cache, void* v_cache,
               const int32_t* page_table, int32_t first_pos, void* scratch, size_t scratch_bytes, void* stream) {
    Dims D;
    if (!make_dims(cfg, &D) || !lw || !h || !k_cache || !v_cache || !page_table || !scratch) return SB_ERR_ARG;
    if (m < 1 || m > SB_MAX_W || first_pos < 0) return SB_ERR_ARG;
    if (first_pos + m > D.max_seq) return SB_ERR_CAPACITY;
    if ((uintptr_t)scratch & 1023) return SB_ERR_ARG;
    if (scratch_bytes < carve(D, nullptr, false, nullptr)) return SB_ERR_CAPACITY;
    const void* ps[9] = {lw->attn_norm, lw->wq, lw->wk, lw->wv, lw->wo, lw->mlp_norm, lw->w_gate, lw->w_up, lw->w_down};
    for (const void* p : ps)
        if (!p || ((uintptr_t)p & 15)) return SB_ERR_ARG;
    std::lock_guard<std::mutex> lock(g_stateless_mu);
    Exec e;
    e.D = D;
    e.st = (cudaStream_t)stream;
    carve(D, (char*)scratch, false, &e.W);
    e.W.page_table = const_cast<int*>(page_table);
    e.W.h = reinterpret_cast<float*>(h);   // rows 0..m-1 of the caller's buffer are the hidden cache
    e.gemm = pick_gemm(D.f32);
    e.plans = &stateless_plans();
    cudaMemsetAsync(e.W.status, 0, 64, e.st);
    if (g_trace) g_tracer.begin(e.st);
    layer_step(e, *lw, k_cache, v_cache, 0, m, first_pos, nullptr);
    g_tracer.end();
    if (e.err) return e.err;
    return cuda_ok(cudaGetLastError());
}

size_t sb_k_rope_table_bytes(const sb_config* cfg) {
    Dims D;
    if (!make_dims(cfg, &D)) return 0;
    return sizeof(float2) * (size_t)D.n_pages * D.page * (D.hd / 2);
}

int sb_k_rope_table(const sb_config* cfg, void* table, size_t table_bytes, void* stream) {
    Dims D;
    if (!make_dims(cfg, &D) || !table || ((uintptr_t)table & 15)) return SB_ERR_ARG;
    if (table_bytes < sizeof(float2) * (size_t)D.n_pages * D.page * (D.hd / 2)) return SB_ERR_CAPACITY;
    launch_rope_table((cudaStream_t)stream, static_cast<float2*>(table), D.n_pages * D.page, D.hd / 2, D.inv_freq);
    return cuda_ok(cudaGetLastError());
}

int sb_k_layer_chain(const sb_config* cfg, const sb_layer_weights* lw, int32_t n_layers, void* h, int32_t m,
                     void* const* k_caches, void* const* v_caches, const int32_t* page_table, int32_t first_pos,
                     const void* rope_table, void* scratch, size_t scratch_bytes, void* stream) {
    Dims D;
    if (!make_dims(cfg, &D) || !lw || !h || !k_caches || !v_caches || !page_table || !scratch) return SB_ERR_ARG;
    if (n_layers < 1 || n_layers > SB_MAX_LAYERS || m < 1 || m > SB_MAX_W || first_pos < 0) return SB_ERR_ARG;
    if (first_pos + m > D.max_seq) return SB_ERR_CAPACITY;
    if (((uintptr_t)scratch & 1023) || ((uintptr_t)rope_table & 15)) return SB_ERR_ARG;
    if (scratch_bytes < carve(D, nullptr, false, nullptr)) return SB_ERR_CAPACITY;
    for (int l = 0; l < n_layers; ++l) {
        const void* ps[11] = {lw[l].attn_norm, lw[l].wq, lw[l].wk, lw[l].wv, lw[l].wo, lw[l].mlp_norm, lw[l].w_gate,
                              lw[l].w_up, lw[l].w_down, k_caches[l], v_caches[l]};
        for (const void* p : ps)
            if (!p || ((uintptr_t)p & 15)) return SB_ERR_ARG;
    }
    std::lock_guard<std::mutex> lock(g_stateless_mu);
    Exec e;
    e.D = D;
    e.st = (cudaStream_t)stream;
    carve(D, (char*)scratch, false, &e.W);
    e.W.page_table = const_cast<int*>(page_table);
    e.W.h = reinterpret_cast<float*>(h);
    e.W.rope_tab = const_cast<float2*>(static_cast<const float2*>(rope_table));
    e.gemm = pick_gemm(D.f32);
    e.plans = &stateless_plans();
    cudaMemsetAsync(e.W.status, 0, 64, e.st);
    for (int l = 0; l < n_layers; ++l)
        layer_step(e, lw[l], k_caches[l], v_caches[l], 0, m, first_pos, l + 1 < n_layers ? lw[l + 1].attn_norm : nullptr);
    if (e.err) return e.err;
    return cuda_ok(cudaGetLastError());
}

int sb_tau_schedule(float alpha, int32_t L, float* out) {
    if (!out || L < 1 || !(alpha >= 0.f)) return SB_ERR_ARG;
    for (int l = 1; l <= L; ++l) out[l - 1] = 1.f + alpha * (1.f - (float)l / (float)L);
    return SB_OK;
}

double sb_model_speedup(int32_t L, double a, int32_t w, int32_t d_max) {
    double num = (double)L * a * (1.0 - std::pow(a, (double)w));
    return num / ((1.0 - a) * ((double)w * d_max + L - d_max));
}

int sb_plan_gemm(int32_t mode, const int32_t* n_rows, int32_t n_mats, int32_t k, int32_t units, int32_t* rows_per_cta,
                 int32_t* k_splits, int32_t* n_items) {
    if (!rows_per_cta || !k_splits || !n_items) return SB_ERR_ARG;
    int R = 0, S = 0, items = 0;
    if (!tc_plan_query(mode, n_rows, n_mats, k, units, &R, &S, &items)) return SB_ERR_ARG;
    *rows_per_cta = R; *k_splits = S; *n_items = items;
    return SB_OK;
}

const char* sb_strerror(int s) {
    switch (s) {
        case SB_OK: return "ok";
        case SB_ERR_ARG: return "bad argument";
        case SB_ERR_STATE: return "call out of order";
        case SB_ERR_CAPACITY: return "capacity exceeded";
        case SB_ERR_CUDA: return "CUDA error";
        case SB_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
        case SB_ERR_UNSUPPORTED: return "unsupported configuration";
        default: return "unknown status";
    }
}

}  // extern "C"
