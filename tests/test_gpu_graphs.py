"""armor_bcd_step replays repeated iterations from a CUDA graph.  The replay enqueues the same kernels with the same
arguments (the iteration index travels through a device counter), so a call with the graph and a call with direct
launches must agree bit for bit: states, masks and every field of every iteration's record."""
import numpy as np
import pytest
import torch

from oracle import armor_oracle as O
from paper_2510_05528_b200 import binding as Bd
from paper_2510_05528_b200 import inputs
from tests.helpers import DEV, dev, host, make

pytestmark = pytest.mark.gpu

TINY = inputs.CONFIGS["tiny"]
MID = TINY.with_(name="mid", d_out=384, d_in=512, d_block=128, n_tokens=6000, chunk_rows=2048, seed=11)

MODES = {
    "full-exact": dict(h_mode=Bd.H_FULL),
    "diag-exact": dict(h_mode=Bd.H_DIAG),
    "diag-adam": dict(h_mode=Bd.H_DIAG, ab_step=Bd.AB_ADAM),
    "full-adam": dict(h_mode=Bd.H_FULL, ab_step=Bd.AB_ADAM),
    "full-2-sweeps": dict(h_mode=Bd.H_FULL, mask_sweeps=2),
    "full-3-groups": dict(h_mode=Bd.H_FULL, mask_groups=3),
    "diag-gd-beta": dict(h_mode=Bd.H_DIAG, ab_step=Bd.AB_GD, s_step=Bd.S_BETA),
}


@pytest.mark.parametrize("mode", sorted(MODES))
@pytest.mark.parametrize("cfg,prec", [(TINY, Bd.PREC_SIMT), (MID, Bd.PREC_FP16X3)], ids=["tiny-simt", "mid-fp16x3"])
def test_graph_replay_is_bit_identical_to_direct_launches(cfg, prec, mode):
    W = inputs.make_weight(cfg)
    H32 = O.gram(inputs.make_activations(cfg)).astype(np.float32)
    Hd, Wd = dev(H32), dev(W)
    out = {}
    for graphs in (False, True):
        ctx = make(cfg, prec, **MODES[mode])
        Bd.armor_use_graphs(ctx.ctx, graphs)
        st = ctx.init(Wd, Hd)
        n0 = ctx.launch_count()
        stats_a = ctx.read_stats(ctx.bcd_step(st, Hd, 0, 9)).copy()       # 1 direct + 8 replayed iterations
        stats_b = ctx.read_stats(ctx.bcd_step(st, Hd, 9, 5)).copy()       # a later call: t_first > 0
        out[graphs] = (host(st.A).copy(), host(st.B).copy(), host(st.S).copy(), host(st.M).copy(), stats_a, stats_b,
                       ctx.launch_count() - n0, ctx.device_status()[:4])
    d, g = out[False], out[True]
    for x, y in zip(d[:4], g[:4]):
        assert np.array_equal(x, y)
    for sa, sb in ((d[4], g[4]), (d[5], g[5])):
        assert sa.tobytes() == sb.tobytes()
    assert d[6] == g[6]                       # the launch count counts replayed launches too
    assert d[7] == g[7] == [0, 0, 0, 0]
    assert d[4]["loss_mask"][-1] < d[4]["loss_start"][0]


def test_a_captured_call_and_timing_fall_back_to_direct_launches():
    """With launch timing on the graph is not used (events cannot be replayed); the results are the same."""
    cfg = MID
    W = inputs.make_weight(cfg)
    H32 = O.gram(inputs.make_activations(cfg)).astype(np.float32)
    Hd, Wd = dev(H32), dev(W)
    ctx = make(cfg, Bd.PREC_FP16X3)
    st = ctx.init(Wd, Hd)
    ctx.bcd_step(st, Hd, 0, 6, want_stats=False)
    ref = host(st.S).copy()
    ctx2 = make(cfg, Bd.PREC_FP16X3)
    Bd.armor_kernel_timing_enable(ctx2.ctx, 2)
    st2 = ctx2.init(Wd, Hd)
    ctx2.bcd_step(st2, Hd, 0, 6, want_stats=False)
    torch.cuda.synchronize()
    t = Bd.armor_kernel_timing(ctx2.ctx)
    assert np.array_equal(host(st2.S), ref)
    assert t["gemm"][0] >= 2 * 6 and t["block_product"][0] > 0 and t["cholesky"][0] == 2 * 6 + 1


@pytest.mark.parametrize("mode", ["full-exact", "full-adam", "full-2-sweeps", "diag-exact"])
def test_replay_in_pieces_around_timed_products_is_bit_identical(mode):
    """With events around the dense products only, the iteration is replayed as graph pieces with the products launched
    directly between them: same results as direct launches, and every product of every iteration is timed."""
    cfg = MID
    W = inputs.make_weight(cfg)
    H32 = O.gram(inputs.make_activations(cfg)).astype(np.float32)
    Hd, Wd = dev(H32), dev(W)
    out = {}
    for graphs in (False, True):
        ctx = make(cfg, Bd.PREC_FP16X3, **MODES[mode])
        Bd.armor_use_graphs(ctx.ctx, graphs)
        Bd.armor_kernel_timing_enable(ctx.ctx, 1)
        st = ctx.init(Wd, Hd)
        n0 = ctx.launch_count()
        stats_a = ctx.read_stats(ctx.bcd_step(st, Hd, 0, 9)).copy()
        stats_b = ctx.read_stats(ctx.bcd_step(st, Hd, 9, 5)).copy()
        torch.cuda.synchronize()
        t = Bd.armor_kernel_timing(ctx.ctx)
        out[graphs] = (host(st.A).copy(), host(st.B).copy(), host(st.S).copy(), host(st.M).copy(), stats_a, stats_b,
                       ctx.launch_count() - n0, ctx.device_status()[:4], t["gemm"][0])
    d, g = out[False], out[True]
    for x, y in zip(d[:4], g[:4]):
        assert np.array_equal(x, y)
    for sa, sb in ((d[4], g[4]), (d[5], g[5])):
        assert sa.tobytes() == sb.tobytes()
    assert d[6] == g[6] and d[8] == g[8]
    if MODES[mode]["h_mode"] == Bd.H_FULL:
        assert g[8] >= 2 * 14
    assert d[7] == g[7] == [0, 0, 0, 0]


@pytest.mark.parametrize("cfg", [MID, MID.with_(name="mid256", d_block=256, d_out=512)], ids=["d_block-128", "d_block-256"])
@pytest.mark.parametrize("mode", ["full-exact", "diag-exact", "full-adam"])
def test_fused_gram_pairs_are_bit_identical_to_separate_launches(cfg, mode):
    """The two per-block Grams of the A-step (shared T) and of the B-step (U with itself and with E H) in one launch each:
    every accumulator sees the same MMAs in the same order, so whole runs agree bit for bit."""
    W = inputs.make_weight(cfg)
    H32 = O.gram(inputs.make_activations(cfg)).astype(np.float32)
    Hd, Wd = dev(H32), dev(W)
    out = {}
    for fused in (False, True):
        ctx = make(cfg, Bd.PREC_FP16X3, **MODES[mode])
        Bd.armor_fuse_grams(ctx.ctx, fused)
        st = ctx.init(Wd, Hd)
        n0 = ctx.launch_count()
        stats = ctx.read_stats(ctx.bcd_step(st, Hd, 0, 6)).copy()
        out[fused] = (host(st.A).copy(), host(st.B).copy(), host(st.S).copy(), host(st.M).copy(), stats,
                      ctx.launch_count() - n0, ctx.device_status()[:4])
    d, g = out[False], out[True]
    for x, y in zip(d[:4], g[:4]):
        assert np.array_equal(x, y)
    assert d[4].tobytes() == g[4].tobytes()
    if mode != "full-adam":
        assert g[5] < d[5]                       # fewer launches
    assert d[6] == g[6] == [0, 0, 0, 0]


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["fp32", "bf16"])
def test_gram_with_overlapped_staging_matches_chunk_by_chunk_calls(dtype):
    """One armor_gram call over several staging chunks stages chunk p + 1 on the context's side stream while chunk p is
    contracted; the contractions keep their order, so H equals, bit for bit, the H of one call per chunk (which runs in
    one stream), and both agree with the fp64 Gram."""
    d_in, rows, chunk = 512, 3 * 16384 + 1000, 16384            # four staging chunks, the last one ragged
    g = torch.Generator(device=DEV); g.manual_seed(5)
    X = (torch.randn(rows, d_in, device=DEV, generator=g) * torch.exp(torch.randn(d_in, device=DEV, generator=g))).to(dtype)
    ctx = Bd.ArmorContext(256, d_in, 128, device=DEV, precision=Bd.PREC_FP16X3)
    H1 = ctx.new_gram(); ctx.gram(X, H1)
    H2 = ctx.new_gram()
    for lo in range(0, rows, chunk):
        ctx.gram(X[lo: lo + chunk], H2)
    torch.cuda.synchronize()
    assert torch.equal(H1, H2)
    ref = O.gram(X.float().cpu().numpy())
    assert np.linalg.norm(host(H1) - ref) <= 2e-5 * np.linalg.norm(ref)
    assert ctx.device_status()[:4] == [0, 0, 0, 0]
