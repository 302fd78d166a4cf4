"""Shared helpers of the GPU parity tests (no method arithmetic here)."""
import numpy as np
import torch

from oracle import armor_oracle as O
from paper_2510_05528_b200 import binding as Bd

DEV = "cuda:0"

# Tolerances (relative Frobenius error against the fp64 oracle):
#   fp32-grade modes (SIMT, FP32X3): the 1e-3 of the benchmark spec;
#   TF32 (one tensor-core pass, operands rounded to 10 mantissa bits, relative rounding 2^-11 = 4.9e-4
#   per operand): GEMM outputs carry ~1e-3, the block solves pass that on to A and B with a small
#   amplification, hence 2e-2 for A, B and 1e-2 for S and the loss.
TOL = {
    Bd.PREC_SIMT: dict(A=1e-3, B=1e-3, S=1e-3, loss=1e-3, margin=1e-5, gram=1e-5),
    Bd.PREC_FP32X3: dict(A=1e-3, B=1e-3, S=1e-3, loss=1e-3, margin=1e-5, gram=1e-4),
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
