"""CPU-only checks of the boundary: the C-ABI library builds and loads, exports every symbol that
include/ssgd.h declares, and its host-only calls (shape validation, hash parameters, workspace
sizing, error strings) behave as documented.  Nothing here launches a kernel."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from oracle import derive_params
from paper_1903_04488_b200 import build as B
from paper_1903_04488_b200 import ssgd as S

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
P = 2**31 - 1


@pytest.fixture(scope="module")
def lib():
    B.build()
    return S.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "ssgd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ssgd_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert len(names) >= 18
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in include/ssgd.h but not exported"
    # and the binding marshals exactly those (plus the two string getters)
    assert set(S.SIGNATURES) | {"ssgd_strerror", "ssgd_last_error"} == set(names)


def test_create_validates_shapes(lib):
    ok = dict(d=100, r=5, c=16, k=10, W=2, seed=1)
    S.Ssgd(**ok)
    for bad in (dict(d=0), dict(d=P), dict(r=0), dict(r=2), dict(r=16), dict(r=17), dict(c=0), dict(c=P),
                dict(k=0), dict(k=101), dict(W=0)):
        kw = dict(ok)
        kw.update(bad)
        with pytest.raises(S.SsgdError) as e:
            S.Ssgd(**kw)
        assert e.value.code == S.EINVAL
    assert lib.ssgd_create(None, 1, 1, 1, 1, 1, 0) == S.EINVAL


@pytest.mark.parametrize("seed", [0, 1, 0x5EED, 2**64 - 1])
def test_hash_parameters_agree_with_the_oracle(lib, seed):
    eng = S.Ssgd(1000, 15, 64, 1, 1, seed)
    got = eng.get_hash_params().numpy()
    want = derive_params(seed, 15).astype(np.int64)
    assert (got == want).all()
    eng.set_hash_params([[1, 0, 1, 0]] * 15)
    assert (eng.get_hash_params().numpy() == np.array([[1, 0, 1, 0]] * 15)).all()
    for bad in ([0, 0, 1, 0], [P, 0, 1, 0], [1, P, 1, 0], [1, 0, 0, 0], [1, 0, 1, P]):
        with pytest.raises(S.SsgdError):
            eng.set_hash_params([bad] * 15)


def test_workspace_bytes(lib):
    d, r, c, k, W = 11_173_962, 5, 262_144, 50_000, 16
    eng = S.Ssgd(d, r, c, k, W, 0)
    n = eng.workspace_bytes(100_000)
    floor = 4 * r * c + 8 * d + 8 * 100_000          # table + estimates + per-coordinate sums + candidates and their sums
    extra = 3 * (d // 8) + 8 * d + (1 << 22)         # three coordinate bitmaps (two of the list selection, one of the
    extra += r * c // 8                              # deferred zero-out), a survivor list with room for every coordinate,
    assert floor + extra <= n <= floor + extra + (1 << 20)   # two 2^19-bin histograms, one bit per bucket
    assert n % 256 == 0
    assert eng.workspace_bytes(200_000) > n
    for bad in (k - 1, d + 1):
        with pytest.raises(S.SsgdError):
            eng.workspace_bytes(bad)


def test_unbound_context_refuses_to_run(lib):
    eng = S.Ssgd(100, 5, 16, 10, 2, 1)
    # device pointers are never touched before the bound-state check
    assert lib.ssgd_step(eng._h, 16, 100, C.c_float(0.9), 20, 16, 16, None) == S.ENOTBOUND
    assert lib.ssgd_exact_topk(eng._h, 16, 20, 16, 16, None) == S.ENOTBOUND
    assert lib.ssgd_unsketch_candidates(eng._h, 16, 20, 16, None, None, None) == S.ENOTBOUND
    assert lib.ssgd_sketch_accumulate(eng._h, 16, 100, C.c_float(0.9), 16, None) == S.ENOTBOUND
    assert lib.ssgd_bind(eng._h, None, None, 100, None, 0, 20) == S.EINVAL
    assert lib.ssgd_bind(eng._h, 4, 16, 100, 256, 1 << 30, 20) == S.EALIGN
    assert lib.ssgd_bind(eng._h, 16, 16, 102, 256, 1 << 30, 20) == S.EALIGN      # ld % 4 != 0
    assert lib.ssgd_bind(eng._h, 16, 16, 96, 256, 1 << 30, 20) == S.EINVAL       # ld < d
    assert lib.ssgd_bind(eng._h, 16, 16, 100, 256, 64, 20) == S.EWORKSPACE
    assert lib.ssgd_flush(eng._h, None) == S.ENOTBOUND
    assert eng.launch_count() == 0


def test_mode_setters_check_their_argument(lib):
    eng = S.Ssgd(100, 5, 16, 10, 2, 1)
    for fn, good, bad in ((lib.ssgd_set_zero_mode, (S.ZERO_DEFERRED, S.ZERO_EAGER), (-1, 2)),
                          (lib.ssgd_set_prune_mode, (S.PRUNE_AUTO, S.PRUNE_OFF, S.PRUNE_ON, S.PRUNE_EARLY_EXIT, S.PRUNE_FUSED), (-1, 5)),
                          (lib.ssgd_set_accumulate_schedule, (S.SCHED_AUTO, S.SCHED_COORDINATE_MAJOR, S.SCHED_WORKER_MAJOR), (-1, 3)),
                          (lib.ssgd_set_insert_mode, (S.INSERT_AUTO, S.INSERT_GLOBAL, S.INSERT_SMEM, S.INSERT_TMA),
                           (-1, 4))):
        for m in good:
            assert fn(eng._h, m) == S.OK
        for m in bad:
            assert fn(eng._h, m) == S.EINVAL
        assert fn(None, good[0]) == S.EINVAL


def test_error_strings(lib):
    seen = set()
    for code in range(0, -9, -1):
        s = lib.ssgd_strerror(code).decode()
        assert s and s != "unknown error"
        seen.add(s)
    assert len(seen) == 9
    assert lib.ssgd_strerror(-99).decode() == "unknown error"


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(S, "_lib", None)
    monkeypatch.setattr(S, "LIB_PATH", str(tmp_path / "libssgd.so"))
    with pytest.raises(RuntimeError, match="missing"):
        S.lib()
