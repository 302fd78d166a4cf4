"""Host-side checks that need no GPU: the shared library loads, exports every symbol the header declares,
and rejects bad arguments before touching the device."""
import ctypes as C
import os
import re

import pytest

from paper_2510_05528_b200 import binding as Bd
from paper_2510_05528_b200 import build as armor_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    armor_build.build()
    return Bd.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "armor.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(armor_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert {"armor_gram", "armor_init", "armor_bcd_step", "armor_proxy_loss", "armor_apply"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n
    assert set(names) == set(Bd.EXPORTS)


def test_config_validation(lib):
    ok = Bd.make_config(256, 256, 32)
    assert Bd.armor_workspace_bytes(ok) > 0
    cases = [
        (Bd.make_config(256, 250, 32), 2),             # d_block does not divide d_in
        (Bd.make_config(256, 256, 30), 2),             # ... nor d_out; not a multiple of m_group either
        (Bd.make_config(256, 256, 32, n_keep=3, m_group=8), 7),      # only 2:4 and 4:8, 5:8, 6:8
        (Bd.make_config(256, 256, 32, n_keep=7, m_group=8), 7),
        (Bd.make_config(256, 256, 32, n_keep=2, m_group=8), 7),
        (Bd.make_config(1024, 1024, 512), 7),          # d_block > 256
        (Bd.make_config(576, 576, 144), 7),            # above 128 the block size must be a multiple of 32
        (Bd.make_config(256, 256, 32, h_mode=5), 1),
        (Bd.make_config(256, 256, 32, select_mode=4), 1),
        (Bd.make_config(256, 256, 32, ab_step=3), 1),
        (Bd.make_config(256, 256, 32, mask_sweeps=65), 1),
        (Bd.make_config(256, 256, 32, mask_sweeps=-1), 1),
        (Bd.make_config(256, 256, 32, mask_groups=9), 1),
        (Bd.make_config(256, 256, 32, ab_step=Bd.AB_ADAM, adam_beta1=1.5), 1),
        (Bd.make_config(256, 256, 32, ab_step=Bd.AB_GD), 7),          # the paper's gradient steps need the diagonal weighting
        (Bd.make_config(256, 256, 32, ridge=-1.0), 1),
        (Bd.make_config(0, 256, 32), 2),
        (Bd.make_config(192, 192, 32, precision=Bd.PREC_TF32), 7),   # tensor-core tiles need multiples of 128
    ]
    for good in (Bd.make_config(256, 256, 32, n_keep=4, m_group=8), Bd.make_config(256, 256, 32, n_keep=5, m_group=8),
                 Bd.make_config(256, 256, 32, n_keep=6, m_group=8), Bd.make_config(512, 512, 256),
                 Bd.make_config(256, 256, 32, s_step=Bd.S_BETA), Bd.make_config(256, 256, 32, mask_sweeps=8), Bd.make_config(256, 256, 32, mask_groups=4),
                 Bd.make_config(256, 256, 32, ab_step=Bd.AB_GD, h_mode=Bd.H_DIAG),
                 Bd.make_config(256, 256, 32, ab_step=Bd.AB_ADAM, adam_lr=1e-3)):
        assert Bd.armor_workspace_bytes(good) > 0
    for cfg, code in cases:
        n = C.c_size_t(0)
        assert lib.armor_workspace_bytes(C.byref(cfg), C.byref(n)) == code
    assert lib.armor_workspace_bytes(None, C.byref(C.c_size_t(0))) == 1
    assert lib.armor_workspace_bytes(C.byref(ok), None) == 1


def test_packed_sizes_and_their_limits(lib):
    """Sizes of the packed core and of the packed layer: kept values (half the entries, bf16), positions (4 bits
    per group of four), and for the layer the bf16 blocks of both wrappers; only 2:4 with 128-aligned shapes."""
    cfg = Bd.make_config(512, 768, 128)
    wn = 512 * 768
    assert Bd.armor_packed_core_bytes(cfg) == wn + wn // 8
    assert Bd.armor_packed_layer_bytes(cfg) == wn + wn // 8 + (512 + 768) * 128 * 2
    n = C.c_size_t(0)
    for bad in (Bd.make_config(512, 768, 128, n_keep=4, m_group=8),     # the sparse tensor cores take 2:4 only
                Bd.make_config(512, 704, 64)):                          # d_in not a multiple of 128
        assert lib.armor_packed_core_bytes(C.byref(bad), C.byref(n)) == 7
        assert lib.armor_packed_layer_bytes(C.byref(bad), C.byref(n)) == 7
    small_blocks = Bd.make_config(512, 768, 64)                         # the core packs, the bf16 wrappers need d_block 128 / 256
    assert lib.armor_packed_core_bytes(C.byref(small_blocks), C.byref(n)) == 0
    assert lib.armor_packed_layer_bytes(C.byref(small_blocks), C.byref(n)) == 7
    assert lib.armor_packed_layer_bytes(None, C.byref(n)) == 1
    assert lib.armor_pack_core(None, None, None, None, None) == 1
    assert lib.armor_apply_layer(None, None, None, None, 4, None) == 1


def test_create_rejects_bad_workspace(lib):
    cfg = Bd.make_config(256, 256, 32)
    ctx = C.c_void_p(0)
    assert lib.armor_create(C.byref(ctx), C.byref(cfg), None, 1 << 30) == 1
    assert lib.armor_create(C.byref(ctx), C.byref(cfg), C.c_void_p(0x1000 + 8), 1 << 30) == 3   # misaligned
    assert lib.armor_create(C.byref(ctx), C.byref(cfg), C.c_void_p(0x1000), 16) == 3           # too small
    assert lib.armor_create(None, C.byref(cfg), C.c_void_p(0x1000), 1 << 30) == 1
    assert ctx.value is None


def test_null_context_is_rejected(lib):
    assert lib.armor_destroy(None) == 1
    assert lib.armor_gram(None, None, 0, 0, 0, None, None) == 1
    assert lib.armor_bcd_step(None, None, None, None, None, None, None, 0, 1, None, None) == 1
    assert lib.armor_proxy_loss(None, None, None, None, None, None, None, None) == 1
    assert lib.armor_apply(None, None, None, None, None, None, None, None, None, 0, 0, None) == 1
    assert lib.armor_launch_count(None) == -1


def test_status_strings(lib):
    seen = {Bd.status_string(i) for i in range(9)}
    assert len(seen) == 9 and "ok" in seen
    assert "unknown" in Bd.status_string(99)


def test_binding_refuses_cpu_tensors(lib):
    import torch
    with pytest.raises(ValueError):
        Bd._ptr(torch.zeros(4), torch.float32, "x")
    with pytest.raises(ValueError):
        Bd.ArmorContext(256, 256, 32, device="cpu")
