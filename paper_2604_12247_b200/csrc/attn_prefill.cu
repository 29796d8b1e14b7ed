// Tiled causal attention of the wide prefill passes (Section 4.3: prefill is the base model's; bf16 models).
//
// A pass carries up to 128 prompt rows per layer.  The decode attention kernel (CUDA cores, one CTA per 128 cached
// positions and block of 8 rows) re-reads and re-unpacks the cached K/V for every block of 8 rows; here a CTA takes a
// tile of 16 prompt rows of ONE query head and walks the cached positions 0 .. (last row's position) in blocks of 64,
// staged once per tile by 16-byte asynchronous copies (three buffers, two blocks in flight), with the two contractions on the tensor cores
// (mma.sync m16n8k16, bf16 x bf16 -> fp32):
//
//   scores   S = Q K^T : Q is fp32; it enters as its high and low bf16 halves (two MMAs), so the product is as
//                        accurate as an fp32 one; K is the cached bf16 row, exact.
//   softmax            : running row maximum / sum in fp32 registers (quad shuffles), flash-attention style
//   out      O += P V  : P enters as high + low bf16 halves (two MMAs), V is the cached bf16 row.
//
// The four warps of a CTA split every 64-position block (16 positions each) and keep separate (max, sum, out) states,
// merged through shared memory at the end.  Output: the bf16 high/low operand rows of the output projection, in the
// block-major layout of the wide GEMMs.  Rows, their rotated queries (fp32) and the pass's K/V rows come from
// k_rope_append, launched before.
#include <cuda_bf16.h>

#include "attn_common.cuh"

namespace sb {

constexpr int kPfRows = 16;          // prompt rows per CTA
constexpr int kPfBlock = 64;         // cached positions per staged block
constexpr int kPfWarps = 4;
constexpr int kPfStages = 3;         // staged blocks in flight per CTA (104 KB at 128 channels: two CTAs per SM)

__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
// x and y as one register of two bf16 (x in the low half): the high parts, and what is left of each as a second register
__device__ __forceinline__ void split_pair(float x, float y, uint32_t& hi, uint32_t& lo) {
    const __nv_bfloat16 hx = __float2bfloat16_rn(x), hy = __float2bfloat16_rn(y);
    const __nv_bfloat16 lx = __float2bfloat16_rn(x - __bfloat162float(hx)), ly = __float2bfloat16_rn(y - __bfloat162float(hy));
    hi = (uint32_t)__bfloat16_as_ushort(hx) | ((uint32_t)__bfloat16_as_ushort(hy) << 16);
    lo = (uint32_t)__bfloat16_as_ushort(lx) | ((uint32_t)__bfloat16_as_ushort(ly) << 16);
}

struct PrefillAttnArgs {
    const float* q;            // [M][H * hd] rotated queries, row i at position pos0 + i
    const __nv_bfloat16* k_cache;   // [n_pages][page][Hkv * hd]
    const __nv_bfloat16* v_cache;
    const int* page_table;
    __nv_bfloat16* act_out;    // [block of 8 rows][16][H * hd]: high halves in rows 0-7, low halves in rows 8-15
    int H, Hkv, page, page_shift;
    int pos0, M;
};

template <int HD>
__global__ void __launch_bounds__(kPfWarps * 32) k_attn_prefill(PrefillAttnArgs a) {
    constexpr int ROWB = HD * 2 + 16;                    // padded row pitch: 8 rows x 16 bytes hit 32 distinct banks
    constexpr int kTile = kPfBlock * ROWB;               // one staged K or V block
    constexpr int KS = HD / 16;                          // k steps of the score contraction
    constexpr int NT = HD / 8;                           // n tiles of the output
    extern __shared__ __align__(16) unsigned char smem[];   // [kPfStages buffers][K block | V block]; reused for the final merge
    pdl_trigger();
    const int h = blockIdx.x, tile = (int)gridDim.y - 1 - (int)blockIdx.y;   // the tiles with the most positions start first
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, tig = lane & 3;
    const int G = a.H / a.Hkv, kvh = h / G;
    const int kvd = a.Hkv * HD, qd = a.H * HD;
    const int row0 = tile * kPfRows;                     // first prompt row of the tile
    const int n_rows = min(kPfRows, a.M - row0);
    const int last_pos = a.pos0 + row0 + n_rows - 1;     // the tile's last row attends over 0 .. last_pos
    const int n_blocks = last_pos / kPfBlock + 1;
    pdl_wait();

    // cached rows blk * 64 .. + 63 of K and V into buffer buf: a thread owns one 16-byte column of pieces and walks the
    // rows; the row's page and offset are computed once and serve both the K and the V copy
    auto stage = [&](int blk, int buf) {
        unsigned char* base = smem + (size_t)buf * 2 * kTile;
        constexpr int kPieces = HD * 2 / 16;                         // 16-byte pieces per row (8 or 16)
        constexpr int kRowsPerSweep = kPfWarps * 32 / kPieces;       // rows the CTA covers per sweep
        const int piece = threadIdx.x % kPieces;
        const unsigned char* kc = reinterpret_cast<const unsigned char*>(a.k_cache) + (size_t)kvh * HD * 2 + piece * 16;
        const unsigned char* vc = reinterpret_cast<const unsigned char*>(a.v_cache) + (size_t)kvh * HD * 2 + piece * 16;
#pragma unroll 4
        for (int r = threadIdx.x / kPieces; r < kPfBlock; r += kRowsPerSweep) {
            const int t = blk * kPfBlock + r;
            unsigned char* dst = base + (size_t)r * ROWB + piece * 16;
            if (t <= last_pos) {
                const int page = a.page_table[t >> a.page_shift];
                const size_t off = ((size_t)page * a.page + (t & (a.page - 1))) * kvd * 2;
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(dst)), "l"(kc + off) : "memory");
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(dst + kTile)), "l"(vc + off) : "memory");
            } else {   // beyond the tile's last position: the probabilities are 0 there, and 0 * garbage must stay 0
                *reinterpret_cast<uint4*>(dst) = make_uint4(0u, 0u, 0u, 0u);
                *reinterpret_cast<uint4*>(dst + kTile) = make_uint4(0u, 0u, 0u, 0u);
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    stage(0, 0);
    if (n_blocks > 1) stage(1, 1);

    // this thread's query fragments: rows g and g + 8 of the tile, high and low halves
    uint32_t qh[KS][4], ql[KS][4];
    {
        const int ra = min(row0 + g, a.M - 1), rb = min(row0 + g + 8, a.M - 1);   // rows past the pass repeat the last one (never stored)
        const float* qa = a.q + (size_t)ra * qd + (size_t)h * HD;
        const float* qb = a.q + (size_t)rb * qd + (size_t)h * HD;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            const float2 a0 = *reinterpret_cast<const float2*>(qa + 16 * ks + 2 * tig);
            const float2 a1 = *reinterpret_cast<const float2*>(qb + 16 * ks + 2 * tig);
            const float2 a2 = *reinterpret_cast<const float2*>(qa + 16 * ks + 8 + 2 * tig);
            const float2 a3 = *reinterpret_cast<const float2*>(qb + 16 * ks + 8 + 2 * tig);
            split_pair(a0.x, a0.y, qh[ks][0], ql[ks][0]);
            split_pair(a1.x, a1.y, qh[ks][1], ql[ks][1]);
            split_pair(a2.x, a2.y, qh[ks][2], ql[ks][2]);
            split_pair(a3.x, a3.y, qh[ks][3], ql[ks][3]);
        }
    }
    const float scale = attn_score_scale(HD);
    const int pos_a = a.pos0 + row0 + g, pos_b = pos_a + 8;   // positions of this thread's two rows
    float m_a = -INFINITY, m_b = -INFINITY, l_a = 0.f, l_b = 0.f;
    float o[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f;

    for (int blk = 0; blk < n_blocks; ++blk) {
        const int buf = blk % kPfStages;
        // two blocks ahead (its buffer was released by the barrier that ended the previous iteration); the copies of
        // a CTA are latency, not bandwidth: the more of them are in flight the better
        if (blk + 2 < n_blocks) {
            stage(blk + 2, (blk + 2) % kPfStages);
            asm volatile("cp.async.wait_group 2;" ::: "memory");
        } else if (blk + 1 < n_blocks) {
            asm volatile("cp.async.wait_group 1;" ::: "memory");
        } else {
            asm volatile("cp.async.wait_group 0;" ::: "memory");
        }
        __syncthreads();                                  // block blk is in place for every warp
        const uint32_t k_s = smem_u32(smem + (size_t)buf * 2 * kTile), v_s = k_s + kTile;
        const int p0 = blk * kPfBlock + warp * 16;        // this warp's 16 positions of the block
        if (p0 <= last_pos) {
            // ---- scores: two n tiles (positions p0 .. p0+7, p0+8 .. p0+15) ----
            // (the high and the low halves of q accumulate separately: four independent chains of MMAs instead of two)
            float s[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
            float sl[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
                // matrices: (positions 0-7, channels lo), (0-7, hi), (8-15, lo), (8-15, hi)
                uint32_t kb[4];
                const int r = warp * 16 + (lane & 7) + ((lane >> 4) << 3), cbyte = (16 * ks + ((lane >> 3) & 1) * 8) * 2;
                ldmatrix_x4(kb, k_s + (uint32_t)(r * ROWB + cbyte));
                mma_bf16(s[0], qh[ks], kb[0], kb[1]);
                mma_bf16(sl[0], ql[ks], kb[0], kb[1]);
                mma_bf16(s[1], qh[ks], kb[2], kb[3]);
                mma_bf16(sl[1], ql[ks], kb[2], kb[3]);
            }
#pragma unroll
            for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                for (int j = 0; j < 4; ++j) s[nt][j] += sl[nt][j];
            // ---- online softmax of rows g (values [.][0], [.][1]) and g + 8 ([.][2], [.][3]) ----
            float mx_a = -INFINITY, mx_b = -INFINITY;
#pragma unroll
            for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                for (int j = 0; j < 2; ++j) {
                    const int t = p0 + nt * 8 + 2 * tig + j;
                    s[nt][j] = t <= pos_a ? s[nt][j] * scale : -INFINITY;
                    s[nt][2 + j] = t <= pos_b ? s[nt][2 + j] * scale : -INFINITY;
                    mx_a = fmaxf(mx_a, s[nt][j]);
                    mx_b = fmaxf(mx_b, s[nt][2 + j]);
                }
            mx_a = fmaxf(mx_a, __shfl_xor_sync(0xffffffffu, mx_a, 1)); mx_a = fmaxf(mx_a, __shfl_xor_sync(0xffffffffu, mx_a, 2));
            mx_b = fmaxf(mx_b, __shfl_xor_sync(0xffffffffu, mx_b, 1)); mx_b = fmaxf(mx_b, __shfl_xor_sync(0xffffffffu, mx_b, 2));
            const float nm_a = fmaxf(m_a, mx_a), nm_b = fmaxf(m_b, mx_b);
            const float f_a = nm_a > -INFINITY ? expf(m_a - nm_a) : 1.f, f_b = nm_b > -INFINITY ? expf(m_b - nm_b) : 1.f;
            float ps_a = 0.f, ps_b = 0.f;
            uint32_t ph[4], pl[4];                         // P as the A operand of the second contraction: k = the 16 positions
            {
                float pv[2][4];
#pragma unroll
                for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                    for (int j = 0; j < 2; ++j) {
                        pv[nt][j] = nm_a > -INFINITY ? expf(s[nt][j] - nm_a) : 0.f;
                        pv[nt][2 + j] = nm_b > -INFINITY ? expf(s[nt][2 + j] - nm_b) : 0.f;
                        ps_a += pv[nt][j];
                        ps_b += pv[nt][2 + j];
                    }
                split_pair(pv[0][0], pv[0][1], ph[0], pl[0]);   // row g,     positions 2 tig, 2 tig + 1
                split_pair(pv[0][2], pv[0][3], ph[1], pl[1]);   // row g + 8
                split_pair(pv[1][0], pv[1][1], ph[2], pl[2]);   // row g,     positions 8 + 2 tig ..
                split_pair(pv[1][2], pv[1][3], ph[3], pl[3]);   // row g + 8
            }
            ps_a += __shfl_xor_sync(0xffffffffu, ps_a, 1); ps_a += __shfl_xor_sync(0xffffffffu, ps_a, 2);
            ps_b += __shfl_xor_sync(0xffffffffu, ps_b, 1); ps_b += __shfl_xor_sync(0xffffffffu, ps_b, 2);
            l_a = l_a * f_a + ps_a; l_b = l_b * f_b + ps_b;
            m_a = nm_a; m_b = nm_b;
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) { o[nt][0] *= f_a; o[nt][1] *= f_a; o[nt][2] *= f_b; o[nt][3] *= f_b; }
            // ---- out += P V: k = the warp's 16 positions, n = 8 channels per tile; V delivered transposed ----
#pragma unroll
            for (int np = 0; np < NT / 2; ++np) {
                // matrices: (positions 0-7, channels c), (8-15, c), (0-7, c + 8), (8-15, c + 8)
                uint32_t vb[4];
                const int r = warp * 16 + (lane & 7) + (((lane >> 3) & 1) << 3), cbyte = (16 * np + (lane >> 4) * 8) * 2;
                ldmatrix_x4_trans(vb, v_s + (uint32_t)(r * ROWB + cbyte));
                mma_bf16(o[2 * np], ph, vb[0], vb[1]);
                mma_bf16(o[2 * np], pl, vb[0], vb[1]);
                mma_bf16(o[2 * np + 1], ph, vb[2], vb[3]);
                mma_bf16(o[2 * np + 1], pl, vb[2], vb[3]);
            }
        }
        __syncthreads();                                  // every warp is done with buffer buf before it is refilled
    }

    // ---- merge the four warps' states: [warp][16 rows][HD + 2] floats over the staging buffers ----
    float* mrg = reinterpret_cast<float*>(smem);
    {
        float* wa = mrg + ((size_t)warp * kPfRows + g) * (HD + 2);
        float* wb = wa + 8 * (HD + 2);
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            *reinterpret_cast<float2*>(wa + nt * 8 + 2 * tig) = make_float2(o[nt][0], o[nt][1]);
            *reinterpret_cast<float2*>(wb + nt * 8 + 2 * tig) = make_float2(o[nt][2], o[nt][3]);
        }
        if (tig == 0) { wa[HD] = m_a; wa[HD + 1] = l_a; wb[HD] = m_b; wb[HD + 1] = l_b; }
    }
    __syncthreads();
    for (int idx = threadIdx.x; idx < n_rows * (HD / 2); idx += blockDim.x) {
        const int r = idx / (HD / 2), e = (idx - r * (HD / 2)) * 2;
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < kPfWarps; ++w) M = fmaxf(M, mrg[((size_t)w * kPfRows + r) * (HD + 2) + HD]);
        float L = 0.f, O0 = 0.f, O1 = 0.f;
#pragma unroll
        for (int w = 0; w < kPfWarps; ++w) {
            const float* src = mrg + ((size_t)w * kPfRows + r) * (HD + 2);
            const float mw = src[HD];
            if (mw > -INFINITY) {
                const float f = expf(mw - M);
                L += src[HD + 1] * f;
                O0 += src[e] * f;
                O1 += src[e + 1] * f;
            }
        }
        const int row = row0 + r, blk8 = row / kMaxW, i = row - blk8 * kMaxW;
        __nv_bfloat16* dst = a.act_out + ((size_t)blk8 * 16 + i) * qd + (size_t)h * HD + e;
        uint32_t hi, lo;
        split_pair(O0 / L, O1 / L, hi, lo);
        *reinterpret_cast<uint32_t*>(dst) = hi;
        *reinterpret_cast<uint32_t*>(dst + (size_t)8 * qd) = lo;
    }
}

// q: [M][H * hd] fp32 (launch_rope_append ran before and appended the pass's K/V rows); act_out: wide operand layout
bool launch_attention_prefill(cudaStream_t st, const float* q, const void* k_cache, const void* v_cache, const int* page_table,
                              void* act_out, int H, int Hkv, int hd, int page, int page_shift, int pos0, int M) {
    if (hd != 64 && hd != 128) return false;
    PrefillAttnArgs a{q, static_cast<const __nv_bfloat16*>(k_cache), static_cast<const __nv_bfloat16*>(v_cache), page_table,
                      static_cast<__nv_bfloat16*>(act_out), H, Hkv, page, page_shift, pos0, M};
    const dim3 grid(H, (M + kPfRows - 1) / kPfRows), block(kPfWarps * 32);
    const size_t smem = (size_t)kPfStages * 2 * kPfBlock * (hd * 2 + 16);
    static bool configured[kMaxDevices][2];
    const int dev = current_device();
    if (dev < 0) return false;
    if (hd == 128) {
        if (!configured[dev][1]) { cudaFuncSetAttribute(k_attn_prefill<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem); configured[dev][1] = true; }
        return launch_kc(k_attn_prefill<128>, grid, block, smem, st, 1, a) == cudaSuccess;
    }
    if (!configured[dev][0]) { cudaFuncSetAttribute(k_attn_prefill<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem); configured[dev][0] = true; }
    return launch_kc(k_attn_prefill<64>, grid, block, smem, st, 1, a) == cudaSuccess;
}

}  // namespace sb
