"""Host-side checks of the C ABI that need no GPU: the library loads, exports
every declared symbol, and rejects bad arguments before touching the device."""
import ctypes as C
import os
import re

import pytest

from paper_2002_09539_b200 import binding
from paper_2002_09539_b200.build import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build()
    return binding.load_library()


def test_every_declared_symbol_is_exported(lib):
    names = set()
    inc = os.path.join(ROOT, "include")
    for fn in os.listdir(inc):
        text = open(os.path.join(inc, fn)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names |= set(re.findall(r"\b(olsgd_[a-z_0-9]+)\s*\(", text))
    assert len(names) >= 14
    for n in sorted(names):
        assert hasattr(lib, n), n


def test_param_count_matches_the_flat_layout(lib):
    P = C.c_int64()
    for kind, dims, want in [("linreg", [64], 64), ("softmax", [3072, 10], 30730),
                             ("mlp", [3072, 1024, 1024, 10], 4206602),
                             ("mlp", [3072, 512, 10], 1578506)]:
        s = binding._spec(kind, dims)
        assert lib.olsgd_param_count(C.byref(s), C.byref(P)) == 0
        assert P.value == want
    s = binding._spec("flat", flat_P=12345)
    assert lib.olsgd_param_count(C.byref(s), C.byref(P)) == 0 and P.value == 12345


def _hp(**kw):
    d = dict(m=4, tau=2, batch=8, gamma=0.1, alpha=0.5, beta=0.0, mu=0.0, seed=0)
    d.update(kw)
    return binding._HParams(d["m"], d["tau"], d["batch"], d.get("mode", 0), d["gamma"], d["alpha"], d["beta"],
                            d["mu"], d["seed"])


@pytest.mark.parametrize("bad", [dict(m=0), dict(tau=0), dict(batch=0), dict(gamma=0.0),
                                 dict(gamma=-1.0), dict(alpha=-0.1), dict(alpha=1.5),
                                 dict(beta=1.0), dict(beta=-0.1), dict(mu=1.0),
                                 dict(gamma=float("nan")), dict(mode=2), dict(mode=-1)])
def test_bad_hyper_parameters_are_rejected(lib, bad):
    s = binding._spec("flat", flat_P=100)
    n = C.c_size_t()
    hp = _hp(**bad)
    assert lib.olsgd_workspace_bytes(C.byref(s), C.byref(hp), C.byref(n)) == 1  # EINVAL
    assert len(lib.olsgd_last_error(None)) > 0


def test_bad_model_specs_are_rejected(lib):
    n = C.c_size_t()
    hp = _hp()
    for s in [binding._spec("flat", flat_P=0), binding._spec("linreg", [0]),
              binding._spec("softmax", [10, 5, 3]), binding._spec("mlp", [10]),
              binding._spec("mlp", [64, 128, 64]),          # 64 classes > limit
              binding._spec("mlp", [64, 10], gemm_bf16=1),        # bf16 GEMMs without a hidden layer
              binding._spec("mlp", [64, 128, 10], gemm_bf16=0)]:  # fp32 hidden layers
        assert lib.olsgd_workspace_bytes(C.byref(s), C.byref(hp), C.byref(n)) == 1
    # every width and batch is taken: what the tensor-core kernels cannot do runs on CUDA cores
    for dims in ([64, 100, 10], [50, 37, 21, 7]):
        for mode in (1, 2, 3):
            s = binding._spec("mlp", dims, gemm_bf16=mode)
            assert lib.olsgd_workspace_bytes(C.byref(s), C.byref(_hp(batch=7)), C.byref(n)) == 0
    bad_kind = binding._spec("flat", flat_P=5)
    bad_kind.kind = 9
    assert lib.olsgd_workspace_bytes(C.byref(bad_kind), C.byref(hp), C.byref(n)) == 1


def test_workspace_size_counts_the_resident_state(lib):
    n = C.c_size_t()
    s = binding._spec("flat", flat_P=1_000_000)
    hp = _hp(m=8, mu=0.9, beta=0.9)
    assert lib.olsgd_workspace_bytes(C.byref(s), C.byref(hp), C.byref(n)) == 0
    # two x buffers + u, each [8][1M] fp32, plus z, v, one scratch row and the two rows of
    # partial worker sums that eight workers are added up in
    want = 3 * 8 * 4_000_000 + 5 * 4_000_000
    assert want <= n.value <= want + 65536
    hp_local = _hp(m=8, mu=0.9, beta=0.9, mode=1)   # Local SGD (Eq. 2): no anchor refresh to feed
    assert lib.olsgd_workspace_bytes(C.byref(s), C.byref(hp_local), C.byref(n)) == 0
    assert want - 2 * 4_000_000 <= n.value <= want - 2 * 4_000_000 + 65536


def test_init_rejects_null_and_small_workspace_without_touching_the_device(lib):
    s = binding._spec("flat", flat_P=100)
    hp = _hp()
    ctx = C.c_void_p()
    assert lib.olsgd_init(C.byref(ctx), C.byref(s), C.byref(hp), None, None, None, 0, None, None) == 1
    assert ctx.value is None
    assert lib.olsgd_init(C.byref(ctx), C.byref(s), C.byref(hp), None, 4096, 4096, 16, None, None) == 3
    assert b"workspace too small" in lib.olsgd_last_error(None)
    assert lib.olsgd_init(C.byref(ctx), C.byref(s), C.byref(hp), None, 4100, 4096, 1 << 20, None, None) == 1
    assert lib.olsgd_destroy(None) == 0
    assert lib.olsgd_local_step(None, None) == 1
    assert lib.olsgd_period_sync(None) == 1


def test_kernel_attributes_are_remembered_per_device(lib):
    # one process may open contexts on several GPUs; "this kernel's shared-memory limit is
    # configured" must be remembered per device, which the library checks on its own table
    assert lib.olsgd_selftest_per_device_table() == 0


def test_epoch_rule_cycle_walk_domain_is_below_four_n(lib):
    # the permutation's domain 2^(2h) must cover n and stay below 4 n: then a pass of the
    # cycle walk lands in [0, n) with probability > 1/4 and fewer than 4 passes are expected,
    # far from the 64 after which the device raises its status word
    for n in list(range(1, 300)) + [1023, 1024, 1025, 5000, 65535, 65536, 65537, 10 ** 6,
                                    2 ** 30 - 1, 2 ** 30, 2 ** 30 + 1, 2 ** 31 - 1]:
        h = lib.olsgd_epoch_rule_half_bits(n)
        assert h >= 1 and n <= 2 ** (2 * h) and (2 ** (2 * h) < 4 * n or n <= 2), (n, h)
    assert lib.olsgd_epoch_rule_half_bits(0) == -1
    assert lib.olsgd_epoch_rule_half_bits(2 ** 31) == -1
