"""Host-side checks that need no GPU: the library loads, exports every symbol
the header declares, validates arguments, and refuses to run without a device."""
import ctypes
import os
import re

import pytest
import torch

import paper_2601_22442_b200 as pkg
from paper_2601_22442_b200 import binding, build, layouts

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build_all()
    return pkg.load()


def header_symbols():
    text = open(os.path.join(ROOT, "include", "asyncmesh.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(asyncmesh_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound(lib):
    names = header_symbols()
    assert "asyncmesh_create" in names and "asyncmesh_step" in names
    assert "asyncmesh_lookahead_weights" in names and "asyncmesh_read_params" in names
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(binding.SIGNATURES) == names


def test_config_struct_matches_header_layout():
    # 8-byte alignment everywhere; a mismatch here would corrupt every create call
    offs = {n: getattr(binding.Config, n).offset for n, _ in binding.Config._fields_}
    assert offs["R"] == 0 and offs["S"] == 4 and offs["stage_numel"] == 8
    assert offs["p"] == 16 and offs["tau"] == 24 and offs["flags"] == 28
    assert offs["ema_beta"] == 32 and offs["lr"] == 40 and offs["weight_decay"] == 72
    assert offs["seed"] == 80 and offs["lookahead_delay"] == 88
    assert offs["device"] == 96 and offs["avg_interval"] == 100 and offs["stream"] == 104
    assert offs["alloc"] == 112 and offs["free"] == 120 and offs["alloc_ctx"] == 128
    assert offs["optimizer"] == 136 and offs["correction"] == 140 and offs["momentum_decay"] == 144
    assert offs["coord_base"] == 152 and ctypes.sizeof(binding.Config) == 160


def _cfg(**over):
    numel = (ctypes.c_uint64 * 2)(1000, 2000)
    c = binding.Config()
    c.R, c.S = 2, 2
    c.stage_numel = ctypes.cast(numel, ctypes.POINTER(ctypes.c_uint64))
    c.p, c.tau, c.ema_beta = 0.05, 1, 0.9
    c.lr, c.beta1, c.beta2, c.eps, c.weight_decay = 3e-4, 0.9, 0.95, 1e-8, 0.1
    c._keep = numel
    for k, v in over.items():
        setattr(c, k, v)
    return c


@pytest.mark.parametrize("over,word", [
    (dict(R=0), "R ="), (dict(R=17), "R ="), (dict(S=0), "S ="), (dict(S=65), "S ="),
    (dict(p=-0.1), "p ="), (dict(p=1.5), "p ="), (dict(p=float("nan")), "p ="),
    (dict(tau=65), "tau"), (dict(ema_beta=1.01), "ema_beta"), (dict(lr=0.0), "lr"),
    (dict(eps=0.0), "eps"), (dict(beta1=1.0), "betas"), (dict(tau=3, avg_interval=2), "avg_interval"),
    (dict(avg_interval=-1), "avg_interval"), (dict(optimizer=2), "optimizer"), (dict(flags=8), "flags"), (dict(flags=2048), "flags"),
    (dict(flags=1024), "RING_AS_EXCHANGED"), (dict(flags=1024 | 16, tau=0), "RING_AS_EXCHANGED"),
    (dict(flags=1024 | 64 | 4), "RING_AS_EXCHANGED"), (dict(flags=1024 | 16 | 256), "RING_AS_EXCHANGED"),
    (dict(flags=16 | 64), "exclude"), (dict(correction=2), "correction"),
    (dict(coord_base=(ctypes.c_uint64 * 1)(6)), "coord_base"),
    (dict(coord_base=(ctypes.c_uint64 * 1)(2 ** 32 - 4)), "coord_base"),
])
def test_create_rejects_bad_arguments_without_touching_a_device(lib, over, word):
    h = ctypes.c_void_p()
    rc = lib.asyncmesh_create(ctypes.byref(_cfg(**over)), ctypes.byref(h))
    assert rc == binding.ERR_INVALID_ARG and not h.value
    assert word in pkg.asyncmesh_last_error()


def test_create_rejects_null_and_zero_sized_stage(lib):
    h = ctypes.c_void_p()
    assert lib.asyncmesh_create(None, ctypes.byref(h)) == binding.ERR_INVALID_ARG
    c = _cfg()
    c._keep[1] = 0
    assert lib.asyncmesh_create(ctypes.byref(c), ctypes.byref(h)) == binding.ERR_INVALID_ARG
    c = _cfg()
    c.stage_numel = None
    assert lib.asyncmesh_create(ctypes.byref(c), ctypes.byref(h)) == binding.ERR_INVALID_ARG


def test_null_handles(lib):
    assert lib.asyncmesh_destroy(None) == 0
    assert lib.asyncmesh_step(None, None) == binding.ERR_INVALID_ARG
    assert lib.asyncmesh_status(None) == binding.ERR_INVALID_ARG
    out = ctypes.c_uint64()
    assert lib.asyncmesh_step_count(None, ctypes.byref(out)) == binding.ERR_INVALID_ARG


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the no-device failure")
def test_no_device_means_failure_not_fallback(lib):
    h = ctypes.c_void_p()
    rc = lib.asyncmesh_create(ctypes.byref(_cfg()), ctypes.byref(h))
    assert rc == binding.ERR_CUDA and not h.value
    assert "no CPU path" in pkg.asyncmesh_last_error()
    with pytest.raises(RuntimeError):
        pkg.AsyncMesh(2, [100], 0.1, 1, 0.9)


def test_workload_layouts():
    w = layouts.workloads()
    assert w["llama125m"]["numel"] == [45814272, 21238272, 21238272, 21239040]
    assert sum(w["llama350m"]["numel"]) == 341099520
    assert sum(w["llama1b"]["numel"]) == 953223168 and len(w["llama1b"]["numel"]) == 8
    assert w["toy"]["numel"] == [1 << 20, 1 << 20]
    with pytest.raises(ValueError):
        layouts.llama_stage_numel(64, 5, 128, 100, 2, True)


def test_product_does_not_import_the_oracle():
    pk = os.path.join(ROOT, "paper_2601_22442_b200")
    for dirpath, _, files in os.walk(pk):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower(), f
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith((".py", ".c")):
            assert "paper_2601_22442_b200" not in open(os.path.join(ROOT, "oracle", f)).read()


def test_paper_schedules():
    from paper_2601_22442_b200 import ema_coefficient, learning_rate
    T = 30000
    # EMA coefficient: 0.5 for 1k iterations, then cosine to 0.01 (Section 3.3)
    assert ema_coefficient(1, T) == 0.5 and ema_coefficient(1000, T) == 0.5
    assert abs(ema_coefficient(T, T) - 0.01) < 1e-12
    mid = 1000 + (T - 1000) // 2
    assert abs(ema_coefficient(mid, T) - 0.255) < 1e-4
    vals = [ema_coefficient(t, T) for t in range(1, T + 1, 97)]
    assert all(a >= b for a, b in zip(vals, vals[1:])) and 0.01 <= min(vals)
    # learning rate: linear warm-up 1e-7 -> 3e-4 over 3k, cosine to 3e-5 (Appendix B.1)
    assert abs(learning_rate(3000, T) - 3e-4) < 1e-15
    assert abs(learning_rate(1500, T) - (1e-7 + (3e-4 - 1e-7) / 2)) < 1e-15
    assert abs(learning_rate(T, T) - 3e-5) < 1e-15
    assert learning_rate(1, T) < 3e-7 and learning_rate(16500, T) == pytest.approx(1.65e-4, rel=1e-3)
