"""The remaining benchmark shapes at their full matrix sizes (Llama-8B MLP pair, Qwen GQA projections, the
70B-scale MLP pair with d_block 256 in 2:4 and 4:8), in the FP32X3 tensor-core mode.  The calibration set is
cut to 16,384 tokens so that the host can generate it in seconds; the matrices, block sizes and group patterns
are the full ones.  Checked per shape: the initial masks on sampled rows against the oracle (byte-exact),
one row-block of the A-step against the oracle where the fp64 Gram fits the host comfortably, and the
properties that hold at any size (monotone loss, tracked loss equals a fresh evaluation, valid N:M masks,
zeros off the mask, no failed block solve)."""
import numpy as np
import pytest
import torch

from oracle import armor_oracle as O
from paper_2510_05528_b200 import binding as Bd
from paper_2510_05528_b200 import inputs
from tests.helpers import DEV, dev, host, rel

pytestmark = pytest.mark.gpu

N_TOKENS = 16384
CASES = [
    ("llama8b_up", 2, 4),
    ("llama8b_down", 2, 4),
    ("qwen_q", 2, 4),
    ("qwen_kv", 2, 4),
    ("mlp70b_up", 2, 4),
    ("mlp70b_up", 4, 8),
    ("mlp70b_down", 2, 4),
]


@pytest.mark.parametrize("name,n_keep,m_group", CASES, ids=[f"{c[0]}-{c[1]}of{c[2]}" for c in CASES])
def test_two_iterations_at_full_matrix_size(name, n_keep, m_group):
    cfg = inputs.CONFIGS[name].with_(n_tokens=N_TOKENS)
    db = cfg.d_block
    ctx = Bd.ArmorContext(cfg.d_out, cfg.d_in, db, device=DEV, precision=Bd.PREC_FP32X3, seed=cfg.seed,
                          n_keep=n_keep, m_group=m_group)
    W = inputs.make_weight(cfg)
    H = ctx.new_gram()
    scales = torch.from_numpy(inputs.channel_scales(cfg))
    for i in range(inputs.n_chunks(cfg)):
        ctx.gram(inputs.activation_chunk(cfg, i, scales).to(DEV), H)
    Wd = dev(W)
    st = ctx.init(Wd, H)
    torch.cuda.synchronize()

    # initial masks on sampled rows, byte-exact against the oracle (the score uses diag(H) only)
    hdiag = torch.diagonal(H).cpu().numpy().astype(np.float64)
    rows = np.random.default_rng(1).choice(cfg.d_out, 24, replace=False)
    oc = O.OracleConfig(db, n_keep=n_keep, m_group=m_group, seed=cfg.seed)
    score = W[rows].astype(np.float64) ** 2 * hdiag[None, :]
    order = np.argsort(-score.reshape(len(rows), -1, m_group), axis=2, kind="stable")[:, :, :n_keep]
    Mref = np.zeros((len(rows), cfg.d_in // m_group, m_group), dtype=bool)
    np.put_along_axis(Mref, order, True, axis=2)
    assert np.array_equal(host(st.M)[rows], O.pack_mask(Mref.reshape(len(rows), cfg.d_in), m_group))

    L_init = ctx.proxy_loss(st, H).item()
    stats = ctx.read_stats(ctx.bcd_step(st, H, 0, 2))
    seq = [L_init]
    for s in stats:
        seq += [s["loss_start"], s["loss_A"], s["loss_B"], s["loss_S"], s["loss_mask"]]
    for a, b in zip(seq, seq[1:]):
        assert b <= a * (1 + 1e-5), seq
    assert seq[-1] < 0.98 * L_init
    assert abs(ctx.proxy_loss(st, H).item() - seq[-1]) / seq[-1] < 1e-3
    assert stats["chol_failed"].sum() == 0
    Mb = host(st.M)
    bits = np.unpackbits(Mb[:, :, None], axis=2)[:, :, 8 - m_group:]
    assert np.all(bits.sum(axis=2) == n_keep) and np.all(Mb < (1 << m_group))
    Mfull = O.unpack_mask(Mb, m_group)
    assert np.all(host(st.S)[~Mfull] == 0.0)
    assert ctx.device_status()[:4] == [0, 0, 0, 0]
    del ctx, st

    if cfg.d_in > 8192:
        return
    # one row-block of the A-step from the initial state against the oracle on its own rows
    ctxA = Bd.ArmorContext(cfg.d_out, cfg.d_in, db, device=DEV, precision=Bd.PREC_FP32X3, seed=cfg.seed,
                           n_keep=n_keep, m_group=m_group, phases=Bd.PHASE_A)
    stA = ctxA.init(Wd, H)
    ctxA.bcd_step(stA, H, 0, 1, want_stats=False)
    Hq = host(H).astype(np.float64)
    i = (cfg.d_out // db) // 2
    r = slice(i * db, (i + 1) * db)
    Wr = W[r].astype(np.float64)
    _, B0, S0, _ = O.init(Wr, Hq, O.OracleConfig(db, n_keep=n_keep, m_group=m_group))
    Ai, failed = O.a_step(Wr, np.eye(db)[None], B0, S0, Hq, oc)
    assert failed == 0 and rel(host(stA.A)[i], Ai[0]) < 1e-3
