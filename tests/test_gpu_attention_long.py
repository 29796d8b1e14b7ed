"""Layer pass against the CPU oracle at the attention geometry and the context lengths of the full-size runs.

The attention grid is what the large workloads launch -- 32 query heads of 128 channels over 32 KV heads (the 7B shape)
or 8 KV heads (the grouped-query Llama-3 shape), contexts of 511 .. 8191 cached positions -- so that every attention
path is compared with the oracle element by element: clusters of 4 to 8 chunk CTAs merging through distributed shared
memory (one-launch attention, up to 1024 positions), the hand-over to the separate RoPE / chunk / merge kernels when
the round's last row needs a 9th chunk of 128 positions, and 16- and 64-chunk contexts.  Only d_model and the FFN
width are cut (512), which keeps the oracle at about a second per case; they size the GEMMs, not the attention grid.

The cached K rows are drawn three times wider than the queries would like (scores with a standard deviation of
about 3.4), so every (row, head) puts most of its probability on a handful of positions scattered over the whole
context: a chunk that is dropped, merged twice or masked wrongly moves the hidden state by far more than the
tolerance.
"""
import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2604_12247_b200 import binding, inputs
from gpu_util import HIDDEN_TOL

pytestmark = pytest.mark.gpu

GEOM_7B = inputs.scaled(inputs.LLAMA2_7B, name="attn-7b-geometry", n_layers=1, d_model=512, d_ffn=512, vocab=64)
GEOM_L3 = inputs.scaled(inputs.LLAMA3_8B, name="attn-l3-geometry", n_layers=1, d_model=512, d_ffn=512, vocab=64)
# three query heads per KV head: a group size that is not a power of two (the kernels' index arithmetic has a fast path
# for powers of two), that no split over several CTAs divides, and that gives a warp more than one sweep at 6-8 rows
GEOM_G3 = inputs.scaled(inputs.LLAMA3_8B, name="attn-3-per-kv-geometry", n_layers=1, d_model=512, d_ffn=512, vocab=64,
                        n_heads=24, n_kv_heads=8)
MAX_SEQ = 8200
PAGE = 64
K_SCALE = 3.0

# (rows, first position).  511/512: the round straddles / starts on the 4th -> 5th chunk boundary; 896: 8 chunks;
# 1016: the last row sits at 1023, the last position the one-launch kernel takes; 1017 with 8 rows, 1023 with 4,
# 1024, 1025: hand-over to the long-context kernels (9 chunks); 1150, 1279, 1404: 10 and 11 chunks, where the
# grouped-query geometry changes how many CTAs share a KV head's query heads; 2048: 17 chunks; 8184: 64 chunks, the
# longest context of the micro-benchmarks
CASES = [(1, 511), (8, 511), (4, 512), (8, 896), (8, 1016), (1, 1023), (8, 1017), (4, 1023), (1, 1024), (8, 1024),
         (4, 1025), (6, 1150), (3, 1279), (5, 1404), (2, 1500), (3, 1790), (1, 2048), (8, 2048), (6, 2500), (5, 4000),
         (4, 8184), (8, 8184), (1, 8191)]


class Geometry:
    """One shape's weights, cached history and oracle, built once and reused by every case."""

    def __init__(self, shape):
        self.shape = shape
        self.w = inputs.make_weights(shape, 21, std=0.05)
        g = torch.Generator().manual_seed(1)
        for lw in self.w["layers"]:
            for k in ("attn_norm", "mlp_norm"):
                lw[k] = (1.0 + 0.2 * torch.randn(shape.d_model, generator=g)).to(lw[k].dtype)
        kvd = shape.n_kv_heads * shape.head_dim
        k_hist, self.v_hist = inputs.make_kv(MAX_SEQ, kvd, 31, shape.dtype)
        self.k_hist = (k_hist.float() * K_SCALE).to(k_hist.dtype)
        self.kvd = kvd
        # the oracle's cache holds the whole history; a case overwrites the rows it appends and puts them back
        self.o = oracle.Oracle(shape, self.w, MAX_SEQ)
        self.k64, self.v64 = self.k_hist.double().numpy(), self.v_hist.double().numpy()
        for p in range(MAX_SEQ):
            self.o.set_kv(1, p, self.k64[p], self.v64[p])
        # the GPU's paged caches with permuted physical pages
        n_pages = (MAX_SEQ + PAGE - 1) // PAGE
        self.perm = torch.randperm(n_pages, generator=torch.Generator().manual_seed(3)).to(torch.int32)
        pos = torch.arange(MAX_SEQ)
        self.phys = self.perm[pos // PAGE].long() * PAGE + pos % PAGE
        dt = inputs.torch_dtype(shape.dtype)
        kc = torch.zeros((n_pages * PAGE, kvd), dtype=dt)
        vc = torch.zeros((n_pages * PAGE, kvd), dtype=dt)
        kc[self.phys] = self.k_hist
        vc[self.phys] = self.v_hist
        self.kc0, self.vc0 = kc.cuda(), vc.cuda()
        self.pt = self.perm.cuda()
        self.cfg = binding.make_config(shape, MAX_SEQ, PAGE)
        self.scratch = binding.KernelScratch(self.cfg)
        self.lw = {k: v.cuda() for k, v in self.w["layers"][0].items()}

    def gpu(self, h, first_pos, pre=None):
        """The layer on rows h at first_pos ..; pre = (K rows, V rows) cached at the positions right before first_pos
        in place of the history (rows an earlier pass appended)."""
        m = h.shape[0]
        kc, vc = self.kc0.clone(), self.vc0.clone()
        # positions from first_pos on are what the pass appends: whatever they held must not matter
        idx = self.phys[first_pos:].cuda()
        kc[idx] = 7.0
        vc[idx] = -7.0
        if pre is not None and len(pre[0]):
            at = self.phys[first_pos - len(pre[0]):first_pos].cuda()
            kc[at] = torch.from_numpy(pre[0]).to(kc.dtype).cuda()
            vc[at] = torch.from_numpy(pre[1]).to(vc.dtype).cuda()
        hg = h.clone().cuda()
        binding.k_layer(self.cfg, self.lw, hg, kc, vc, self.pt, first_pos, self.scratch)
        torch.cuda.synchronize()
        new = self.phys[first_pos:first_pos + m].cuda()
        return hg.cpu().numpy(), kc[new].float().cpu().numpy(), vc[new].float().cpu().numpy()

    def ref(self, h, first_pos):
        m = h.shape[0]
        out = self.o.layer_forward(1, h.double().numpy(), first_pos)
        kv = [self.o.get_kv(1, p) for p in range(first_pos, first_pos + m)]
        for p in range(first_pos, min(first_pos + m, MAX_SEQ)):      # put the history back
            self.o.set_kv(1, p, self.k64[p], self.v64[p])
        return out, np.stack([k for k, _ in kv]), np.stack([v for _, v in kv])


@pytest.fixture(scope="module", params=[GEOM_7B, GEOM_L3, GEOM_G3], ids=lambda s: s.name)
def geometry(request):
    g = Geometry(request.param)
    yield g
    g.o.close()


def test_full_geometry_layer_matches_oracle_at_every_attention_path(geometry):
    g = geometry
    shape = g.shape
    worst, sens = 0.0, 1e9
    binding.set_default_gemm(1)              # the TMA + tcgen05 path of the full-size runs
    try:
        for m, first_pos in CASES:
            h = inputs.make_hidden(m, shape.d_model, 11 * m + first_pos)
            got_h, got_k, got_v = g.gpu(h, first_pos)
            ref_h, ref_k, ref_v = g.ref(h, first_pos)
            scale = np.abs(ref_h).max()
            err = np.abs(got_h - ref_h).max() / scale
            worst = max(worst, err)
            assert err < HIDDEN_TOL["bf16"], (shape.name, m, first_pos, err)
            # what the layer adds to a row is of the row's own size: the comparison is not dominated by the residual
            sens = min(sens, np.abs(ref_h - h.numpy()).max() / scale)
            ulp = 2.0 ** -7
            for got, ref in ((got_k, ref_k), (got_v, ref_v)):      # appended rows: within one bf16 step
                assert np.all(np.abs(got - ref) <= ulp * np.abs(ref) + 1e-5), (shape.name, m, first_pos)
    finally:
        binding.set_default_gemm(-1)
    print(f"\n[{shape.name}] {len(CASES)} cases up to {max(p + m for m, p in CASES)} positions: worst relative hidden "
          f"error {worst:.2e} (bound {HIDDEN_TOL['bf16']:.0e}); smallest layer update / hidden scale {sens:.2f}")
    assert sens > 0.2


def test_dropping_one_chunk_would_be_seen(geometry):
    """The comparison above is only worth its tolerance if a chunk-sized mistake exceeds it: recompute one case with
    the oracle blind to one 128-position chunk and require the hidden state to move by far more than the tolerance."""
    g = geometry
    m, first_pos = 8, 2048
    h = inputs.make_hidden(m, g.shape.d_model, 11 * m + first_pos)
    ref_h, _, _ = g.ref(h, first_pos)
    lo = 9 * 128
    for p in range(lo, lo + 128):            # zero K rows score 0 against peaks of about +10: the chunk gets no probability
        g.o.set_kv(1, p, np.zeros_like(g.k64[p]), g.v64[p])
    blind_h, _, _ = g.ref(h, first_pos)
    for p in range(lo, lo + 128):
        g.o.set_kv(1, p, g.k64[p], g.v64[p])
    moved = np.abs(blind_h - ref_h).max() / np.abs(ref_h).max()
    print(f"\n[{g.shape.name}] hiding one chunk of 128 positions moves the hidden state by {moved:.2e}")
    assert moved > 5 * HIDDEN_TOL["bf16"]


@pytest.mark.parametrize("first_pos", [1021, 1405, 2050])
def test_long_context_rows_do_not_depend_on_companions(geometry, first_pos):
    """Row i of a 6-row pass is bit-identical to the same row run alone once the earlier rows' K,V are cached, also
    where the pass straddles the hand-over between the attention kernels (1021: rows at 1021 .. 1023 alone go through
    the 8-chunk clusters, in company through the two-launch kernels), where the number of rows changes how a KV head's
    query heads are spread over CTAs (a row alone and in a pass of six), and deep inside a long context: what
    makes speculative decoding return exactly the autoregressive tokens at any length."""
    g = geometry
    m = 6
    h = inputs.make_hidden(m, g.shape.d_model, 5 + first_pos)
    binding.set_default_gemm(1)
    try:
        all_h, all_k, all_v = g.gpu(h, first_pos)
        for i in range(m):
            one_h, one_k, one_v = g.gpu(h[i:i + 1], first_pos + i, pre=(all_k[:i], all_v[:i]))
            assert np.array_equal(one_h[0], all_h[i]), (g.shape.name, first_pos, i)
            assert np.array_equal(one_k[0], all_k[i]) and np.array_equal(one_v[0], all_v[i])
    finally:
        binding.set_default_gemm(-1)
