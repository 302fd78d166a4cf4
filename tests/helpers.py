"""Shared helpers of the GPU parity tests (no method arithmetic here)."""
import numpy as np
import torch

from oracle import armor_oracle as O
from paper_2510_05528_b200 import binding as Bd

DEV = "cuda:0"

# Tolerances (relative Frobenius error against the fp64 oracle):
#   fp32-grade modes (SIMT, FP32X3): 1e-3, the bound this library is specified to (fp32 results against fp64);
#   FP16X3 carries the same 22 operand bits as FP32X3 (exact power-of-two scaling, two fp16 parts): same bars;
#   TF32 (one tensor-core pass, operands rounded to 10 mantissa bits, relative rounding 2^-11 = 4.9e-4
#   per operand): GEMM outputs carry ~1e-3, the block solves pass that on to A and B with a small
#   amplification, hence 2e-2 for A, B and 1e-2 for S and the loss.
TOL = {
    Bd.PREC_SIMT: dict(A=1e-3, B=1e-3, S=1e-3, loss=1e-3, margin=1e-5, gram=1e-5),
    Bd.PREC_FP32X3: dict(A=1e-3, B=1e-3, S=1e-3, loss=1e-3, margin=1e-5, gram=1e-4),
    Bd.PREC_FP16X3: dict(A=1e-3, B=1e-3, S=1e-3, loss=1e-3, margin=1e-5, gram=1e-4),
    Bd.PREC_TF32: dict(A=2e-2, B=2e-2, S=1e-2, loss=1e-2, margin=2e-2, gram=5e-3),
}


def rel(a, b):
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


def dev(x, dtype=torch.float32):
    return torch.from_numpy(np.ascontiguousarray(x)).to(dtype).to(DEV)


def host(t):
    return t.detach().cpu().numpy()


def load_state(st, A, B, S, M, m_group=4):
    """Copies an oracle state (fp64 arrays, boolean mask) into the GPU state tensors."""
    st.A.copy_(dev(A))
    st.B.copy_(dev(B))
    st.S.copy_(dev(S))
    st.M.copy_(torch.from_numpy(O.pack_mask(M, m_group)).to(DEV))


def mask_block_diffs(Mg_packed, M_oracle, d_block, m_group=4):
    """Set of (i, j) blocks in which the GPU mask differs from the oracle's."""
    diff = Mg_packed != O.pack_mask(M_oracle, m_group)
    rows, cgs = np.nonzero(diff)
    return {(int(r) // d_block, int(c) * m_group // d_block) for r, c in zip(rows, cgs)}


def excused_blocks(info, margin):
    """Blocks whose selection or mask decision was closer than the margin (several answers are valid)."""
    close = (info.select_margin <= margin) | (info.mask_margin <= margin)
    return {(int(i), int(j)) for i, j in zip(*np.nonzero(close))}


def make(cfg, precision, h_mode=Bd.H_FULL, **kw):
    return Bd.ArmorContext(cfg.d_out, cfg.d_in, cfg.d_block, device=DEV, precision=precision, h_mode=h_mode,
                           seed=cfg.seed, **kw)


def run_teacher_forced(cfg, W, H32, prec, h_mode, n_steps, select=Bd.SELECT_L1_RANDOM, n_keep=2, m_group=4,
                       s_step=Bd.S_EXACT, tol_scale=1.0, ab_step=Bd.AB_EXACT):
    ctx = make(cfg, prec, h_mode, select_mode=select, n_keep=n_keep, m_group=m_group, s_step=s_step, ab_step=ab_step)
    Hd = dev(H32)
    st = ctx.init(dev(W), Hd)
    oc = O.OracleConfig(cfg.d_block, h_mode=h_mode, seed=cfg.seed, select_mode=select, n_keep=n_keep,
                        m_group=m_group, s_step=s_step, ab_step=ab_step)
    Hq = H32.astype(np.float64)
    Hw = O.weighting(Hq, h_mode)
    Wn = W.astype(np.float64)
    A, B, S, M = O.init(Wn, Hq, oc)
    tol = {k: v * tol_scale for k, v in TOL[prec].items()}
    n_excused = 0
    worst = dict(A=0.0, B=0.0, S=0.0, loss=0.0)
    for t in range(n_steps):
        load_state(st, A, B, S, M, m_group)        # the GPU starts every step from the oracle's state
        stats = ctx.bcd_step(st, Hd, t, 1)
        sg = ctx.read_stats(stats)[0]
        A, B, S, M, info = O.bcd_iteration(Wn, A, B, S, M, Hw, oc, t)
        worst["A"] = max(worst["A"], rel(host(st.A), A))
        worst["B"] = max(worst["B"], rel(host(st.B), B))
        for k_gpu, k_or in (("loss_start", "start"), ("loss_A", "A"), ("loss_B", "B"), ("loss_S", "S")):
            worst["loss"] = max(worst["loss"], abs(sg[k_gpu] - info.loss[k_or]) / info.loss[k_or])
        assert abs(sg["tau_B"] - info.tau_B) <= 10 * tol["B"] * abs(info.tau_B) + 1e-6
        assert abs(sg["tau_S"] - info.tau_S) <= 10 * tol["S"] * abs(info.tau_S) + 1e-12
        assert sg["chol_failed"] == info.chol_failed == 0
        # masks: identical outside blocks whose decision margin is below the threshold
        diff = mask_block_diffs(host(st.M), M, cfg.d_block, m_group)
        excused = excused_blocks(info, tol["margin"])
        guard_close = abs(info.delta_L_mask) <= tol["margin"] * info.loss["S"]
        if sg["mask_accepted"] != info.mask_accepted:
            assert guard_close, "accept/reject differs although the guard was not marginal"
            n_excused += len(diff)
            continue
        assert diff <= excused, f"step {t}: masks differ in blocks {sorted(diff - excused)} with a clear margin"
        n_excused += len(diff)
        if not diff:
            worst["S"] = max(worst["S"], rel(host(st.S), S))
            assert sg["groups_changed"] == info.groups_changed
            worst["loss"] = max(worst["loss"], abs(sg["loss_mask"] - info.loss["mask"]) / info.loss["mask"])
    assert ctx.device_status()[:4] == [0, 0, 0, 0]
    for k in worst:
        assert worst[k] < tol[k], (k, worst)
    return worst, n_excused
