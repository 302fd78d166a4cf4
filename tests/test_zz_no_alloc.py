"""The no-allocation normalisation entry point (fixed scratch array inside the library), called through the
C ABI, against armor_init's normalisation and against the CPU oracle's.  Collected last on purpose: a failure
here cannot hide another test.

Who needs this call: code that must not obtain device memory when it runs -- the GPU's memory already belongs
to another pool, or the host application forbids allocations after start-up.  So the test hands in buffers it
made beforehand and the call itself allocates nothing."""
import ctypes as C

import numpy as np
import pytest
import torch

from oracle import armor_oracle as O
from paper_2510_05528_b200 import binding as Bd
from tests.helpers import DEV, host

pytestmark = pytest.mark.gpu


def reference_normalisation(W_d):
    """The existing path: armor_init with cfg.normalize = 1 (context + workspace)."""
    d_out, d_in = W_d.shape
    ctx = Bd.ArmorContext(d_out, d_in, 32, device=DEV, precision=Bd.PREC_SIMT, normalize=1)
    H = torch.eye(d_in, dtype=torch.float32, device=DEV)
    st = ctx.init(W_d, H)
    torch.cuda.synchronize()
    return host(st.Wbar).copy(), host(st.r1).copy(), host(st.r2).copy()


def test_no_alloc_normalisation_matches_armor_init_twice_in_a_row():
    rng = np.random.default_rng(21)
    shapes = [(256, 512), (96, 160)]          # the second call is smaller: stale scratch from the first must not matter
    for k, (d_out, d_in) in enumerate(shapes):
        W = (rng.standard_normal((d_out, d_in)) * 0.02).astype(np.float32)
        W[:, 3] = 0.0                          # a dead column and a dead row: norms read as 1
        W[5, :] = 0.0
        W_d = torch.from_numpy(W).to(DEV)
        Wbar = torch.full((d_out, d_in), float("nan"), device=DEV)
        r1 = torch.full((d_in,), float("nan"), device=DEV)
        r2 = torch.full((d_out,), float("nan"), device=DEV)
        if k == 0:
            # module load and the look-up of the scratch array's address happen on a device's first call
            Bd.armor_normalize_noalloc(W_d, Wbar, r1, r2)
            Wbar.fill_(float("nan")); r1.fill_(float("nan")); r2.fill_(float("nan"))
        torch.cuda.synchronize()
        # free device memory as the driver reports it: an allocation by the library (which torch's own counters
        # would not see) lowers it
        free_before, _ = torch.cuda.mem_get_info(DEV)
        torch_before = torch.cuda.memory_allocated(DEV)
        Bd.armor_normalize_noalloc(W_d, Wbar, r1, r2)
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info(DEV)
        assert free_after >= free_before and torch.cuda.memory_allocated(DEV) == torch_before
        Wn_or, r1_or, r2_or = O.normalize(W)
        for got, want in ((Wbar, Wn_or), (r1, r1_or), (r2, r2_or)):
            assert np.linalg.norm(host(got).astype(np.float64) - want) <= 1e-6 * np.linalg.norm(want)
        Wb_ref, r1_ref, r2_ref = reference_normalisation(W_d)
        for got, want in ((Wbar, Wb_ref), (r1, r1_ref), (r2, r2_ref)):
            g = host(got)
            assert np.all(np.isfinite(g))
            assert np.linalg.norm(g.astype(np.float64) - want) <= 1e-6 * np.linalg.norm(want)
        assert host(r1)[3] == 1.0 and host(r2)[5] == 1.0


def test_no_alloc_rejects_sizes_beyond_its_scratch_and_bad_arguments():
    L = Bd.lib()
    W = torch.zeros(8, 8, device=DEV)
    p = C.c_void_p(W.data_ptr())
    assert L.armor_normalize_noalloc(p, 8, 8192 + 1, p, p, p, None) == 8
    assert L.armor_normalize_noalloc(p, 65536 + 1, 8, p, p, p, None) == 8
    assert "scratch" in Bd.status_string(8)
    assert L.armor_normalize_noalloc(None, 8, 8, p, p, p, None) == 1
    assert L.armor_normalize_noalloc(p, 0, 8, p, p, p, None) == 2
