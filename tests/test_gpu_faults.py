"""Failure detection without a GPU fault: a bounded wait that is made to run out, and inputs the method cannot
use (NaN / Inf in W or H, a negative diagonal entry of H) or can use but should report (a dead channel).  Every
case is produced on the host; the device only ever sees ordinary launches."""
import numpy as np
import pytest
import torch

from oracle import armor_oracle as O
from paper_2510_05528_b200 import binding as Bd
from paper_2510_05528_b200 import inputs
from tests.helpers import DEV, TOL, dev, host, load_state, make, rel

pytestmark = pytest.mark.gpu

TINY = inputs.CONFIGS["tiny"]
MID = TINY.with_(name="mid", d_out=384, d_in=512, d_block=128, n_tokens=6000, chunk_rows=2048, seed=11)
ST_TIMEOUTS, ST_LAST, ST_BAD_W, ST_BAD_H, ST_NEG, ST_DEAD, ST_POISON = 2, 3, 5, 6, 7, 8, 9
ERR_INVALID_ARG, ERR_TIMEOUT = 1, 6


def data(cfg):
    W = inputs.make_weight(cfg)
    X = inputs.make_activations(cfg)
    return W, X, O.gram(X).astype(np.float32)


def test_a_wait_that_runs_out_is_reported_and_the_context_stays_usable():
    W, X, H32 = data(MID)
    ctx = make(MID, Bd.PREC_FP16X3)
    Hd = dev(H32)
    st = ctx.init(dev(W), Hd)
    before = ctx.proxy_loss(st, Hd).item()
    res = torch.full((2,), -1, dtype=torch.int32, device=DEV)
    Bd.armor_selftest_wait_timeout(ctx.ctx, 200_000, res)          # about 0.1 ms of spinning
    status = ctx.device_status()
    assert res.tolist() == [0, 1]                                  # gave up; the abort flag is up
    assert status[ST_TIMEOUTS] == 1 and status[ST_LAST] == ERR_TIMEOUT
    Bd.armor_selftest_wait_timeout(ctx.ctx, 1000, res)
    assert ctx.device_status()[ST_TIMEOUTS] == 2
    # the tensor-core kernels (which share the wait routine and the status words) still run and agree
    assert ctx.proxy_loss(st, Hd).item() == before
    sg = ctx.read_stats(ctx.bcd_step(st, Hd, 0, 1))[0]
    assert sg["loss_mask"] < sg["loss_start"] and ctx.device_status()[ST_TIMEOUTS] == 2
    with pytest.raises(Bd.ArmorError):
        Bd.armor_selftest_wait_timeout(ctx.ctx, 0, res)


@pytest.mark.parametrize("cfg,prec", [(TINY, Bd.PREC_SIMT), (MID, Bd.PREC_FP16X3), (MID, Bd.PREC_FP32X3)],
                         ids=["tiny-simt", "mid-fp16x3", "mid-fp32x3"])
def test_unusable_inputs_are_counted_and_every_update_is_withheld(cfg, prec):
    W, X, H32 = data(cfg)
    ctx = make(cfg, prec)
    Hd, Wd = dev(H32), dev(W)
    st = ctx.init(Wd, Hd)
    ctx.bcd_step(st, Hd, 0, 1, want_stats=False)                   # a state away from the initialisation
    keep = [host(t).copy() for t in (st.A, st.B, st.S, st.M)]
    assert ctx.device_status()[ST_BAD_W:ST_POISON + 1] == [0, 0, 0, 0, 0]

    def unchanged():
        return all(np.array_equal(host(t), k) for t, k in zip((st.A, st.B, st.S, st.M), keep))

    # one NaN in W
    Wbad = W.copy(); Wbad[3, 7] = np.nan
    st.Wbar.copy_(dev(Wbad))
    sg = ctx.read_stats(ctx.bcd_step(st, Hd, 1, 2))
    s = ctx.device_status()
    assert unchanged() and s[ST_BAD_W] == 1 and s[ST_POISON] == 1 and s[ST_LAST] == ERR_INVALID_ARG
    assert int(sg["mask_accepted"].sum()) == 0 and int(sg["groups_changed"].sum()) == 0
    assert float(sg["tau_B"].max()) == 0.0 and float(sg["tau_S"].max()) == 0.0
    st.Wbar.copy_(Wd)
    # Inf in H (two entries: the matrix is symmetric)
    Hbad = H32.copy(); Hbad[5, 9] = Hbad[9, 5] = np.inf
    ctx.bcd_step(st, dev(Hbad), 1, 1, want_stats=False)
    s = ctx.device_status()
    assert unchanged() and s[ST_BAD_H] == 2 and s[ST_BAD_W] == 1 and s[ST_POISON] == 1
    # a negative diagonal entry: not a Gram matrix
    Hneg = H32.copy(); Hneg[11, 11] = -Hneg[11, 11]
    ctx.bcd_step(st, dev(Hneg), 1, 1, want_stats=False)
    s = ctx.device_status()
    assert unchanged() and s[ST_NEG] == 1 and s[ST_POISON] == 1
    # clean inputs again: the same context carries on and follows the oracle
    A, B, S = (k.astype(np.float64) for k in keep[:3])
    M = O.unpack_mask(keep[3])
    oc = O.OracleConfig(cfg.d_block, seed=cfg.seed)
    A1, B1, S1, M1, info = O.bcd_iteration(W.astype(np.float64), A, B, S, M, H32.astype(np.float64), oc, 1)
    sg = ctx.read_stats(ctx.bcd_step(st, Hd, 1, 1))[0]
    s = ctx.device_status()
    assert s[ST_POISON] == 0 and s[ST_BAD_W] == 1 and s[ST_BAD_H] == 2 and s[ST_NEG] == 1
    tol = TOL[prec]
    assert rel(host(st.A), A1) < tol["A"] and rel(host(st.B), B1) < tol["B"]
    assert abs(sg["loss_S"] - info.loss["S"]) / info.loss["S"] < tol["loss"]
    # armor_init screens its inputs as well
    ctx.init(dev(Wbad), Hd)
    assert ctx.device_status()[ST_BAD_W] == 2


def test_a_dead_channel_is_reported_and_handled():
    """A channel that is zero on every calibration token: row and column of H vanish.  Legal input (the channel
    carries no weight): counted in its status word, no block solve fails, and the iteration follows the oracle."""
    cfg = MID
    W = inputs.make_weight(cfg)
    X = inputs.make_activations(cfg).copy()
    X[:, 37] = 0.0
    H32 = O.gram(X).astype(np.float32)
    ctx = make(cfg, Bd.PREC_FP16X3)
    Hd = dev(H32)
    st = ctx.init(dev(W), Hd)
    oc = O.OracleConfig(cfg.d_block, seed=cfg.seed)
    Wn, Hq = W.astype(np.float64), H32.astype(np.float64)
    A, B, S, M = O.init(Wn, Hq, oc)
    assert np.array_equal(host(st.M), O.pack_mask(M))
    sg = ctx.read_stats(ctx.bcd_step(st, Hd, 0, 1))[0]
    A, B, S, M, info = O.bcd_iteration(Wn, A, B, S, M, Hq, oc, 0)
    s = ctx.device_status()
    assert s[ST_DEAD] == 1 and s[ST_POISON] == 0 and s[0] == 0 and sg["chol_failed"] == info.chol_failed == 0
    tol = TOL[Bd.PREC_FP16X3]
    assert rel(host(st.A), A) < tol["A"] and rel(host(st.B), B) < tol["B"]
    for k_gpu, k_or in (("loss_start", "start"), ("loss_A", "A"), ("loss_B", "B"), ("loss_S", "S")):
        assert abs(sg[k_gpu] - info.loss[k_or]) / info.loss[k_or] < tol["loss"]


@pytest.mark.parametrize("prec", [Bd.PREC_SIMT, Bd.PREC_FP16X3], ids=["simt", "fp16x3"])
def test_a_diagonal_block_of_H_that_is_not_positive_definite_is_skipped(prec):
    """H with a positive diagonal but an indefinite diagonal block (one off-diagonal pair pushed beyond the
    Cauchy-Schwarz bound): the screening lets it pass, the B-step finds (H_jj + mu I) not positive definite, leaves
    that block of B where it was, counts the failure in every iteration, and moves the other blocks like the
    oracle (B-step alone; its per-call inverse of H_jj is the object under test)."""
    cfg = MID
    W, X, H32 = data(cfg)
    db = cfg.d_block
    j, a, b = 2, 2 * db + 5, 2 * db + 40
    H32 = H32.copy()
    H32[a, b] = H32[b, a] = 1.5 * np.sqrt(H32[a, a] * H32[b, b])
    ctx = make(cfg, prec, phases=Bd.PHASE_B)
    Hd = dev(H32)
    st = ctx.init(dev(W), Hd)
    oc = O.OracleConfig(db, seed=cfg.seed, phases=O.PH_B)
    Wn, Hq = W.astype(np.float64), H32.astype(np.float64)
    A, B, S, M = O.init(Wn, Hq, oc)
    rng = np.random.default_rng(5)
    A = (A + 0.05 * rng.standard_normal(A.shape)).astype(np.float32).astype(np.float64)
    B = (B + 0.05 * rng.standard_normal(B.shape)).astype(np.float32).astype(np.float64)
    load_state(st, A, B, S, M)
    sg = ctx.read_stats(ctx.bcd_step(st, Hd, 0, 2))
    s = ctx.device_status()
    assert [int(x) for x in sg["chol_failed"]] == [1, 1] and s[0] == 2 and s[1] == j + 1 and s[ST_POISON] == 0
    assert np.array_equal(host(st.B)[j], B[j].astype(np.float32))              # the failing block did not move
    B1, tau1, failed1 = O.b_step(Wn, A, B, S, Hq, oc)
    B2, tau2, failed2 = O.b_step(Wn, A, B1, S, Hq, oc)
    assert failed1 == failed2 == 1
    tol = TOL[prec]
    assert abs(sg["tau_B"][0] - tau1) <= 10 * tol["B"] * abs(tau1) and abs(sg["tau_B"][1] - tau2) <= 10 * tol["B"] * abs(tau2)
    assert rel(host(st.B), B2) < tol["B"]


def test_fp16_mode_reports_an_H_outside_its_range_and_passes_nan_activations_on():
    """The three-pass fp16 mode scales H by its diagonal; a positive semidefinite H then fits the fp16 range.  An
    entry far beyond the Cauchy-Schwarz bound does not: it is clamped and counted in status word 10.  A NaN in the
    activations must reach the Gram (and from there the screening), not be swallowed by the clamping."""
    cfg = MID
    W, X, H32 = data(cfg)
    ctx = make(cfg, Bd.PREC_FP16X3)
    H_bad = H32.copy()
    a, b = 7, 300
    H_bad[a, b] = H_bad[b, a] = 100.0 * np.sqrt(H32[a, a] * H32[b, b])
    Hd = dev(H_bad)
    st = ctx.init(dev(W), Hd)
    ctx.proxy_loss(st, Hd)
    assert ctx.device_status()[10] == 2
    Xn = X.copy()
    Xn[17, 5] = np.nan
    H = ctx.new_gram()
    ctx.gram(dev(Xn), H)
    Hh = host(H)
    assert np.isnan(Hh[5, 5]) and np.isnan(Hh[5, 9]) and np.isnan(Hh[9, 5]) and np.isfinite(Hh[9, 9])
    ctx.init(dev(W), H)
    assert ctx.device_status()[ST_BAD_H] >= 2 * cfg.d_in - 1
