"""GPU parity of ssgd_heavymix (Algorithm 1) against the oracle, on the oracle's own fp32 table so that
every decision has identical inputs on both sides: the chosen index set, its exact values and |H| must
then agree exactly, the squared-norm estimate up to the order of its fp64 summation."""
import numpy as np
import pytest
import torch

from oracle import Oracle
from paper_1903_04488_b200 import ssgd as S
from paper_1903_04488_b200 import workloads as wl

pytestmark = pytest.mark.gpu

CASES = [
    (wl.C1.scaled(d=200_001, c=4096, ncand=400, k=400), "planted"),     # planted heavy coordinates + fill
    (wl.C2.scaled(d=150_003, W=3, c=2048, ncand=300, k=300), "plain"),  # nothing or little heavy: mostly fill
    (wl.C3.scaled(d=60_000, W=2, r=7, c=999, ncand=64, k=64), "plain"), # r = 7, c not a power of two
    (wl.C2.scaled(d=5_000, W=2, r=1, c=16, ncand=50, k=50), "plain"),   # one row, many collisions: |H| > k possible
    (wl.C2.scaled(d=33, W=1, r=3, c=8, ncand=7, k=7), "zero"),          # all-zero table: everything is "heavy"
]


@pytest.mark.parametrize("cfg,kind", CASES, ids=lambda x: f"{x.name}-d{x.d}-r{x.r}-c{x.c}-k{x.k}" if hasattr(x, "name") else x)
def test_heavymix_matches_oracle(cuda_device, cfg, kind):
    dev = cuda_device
    eng = S.Ssgd(cfg.d, cfg.r, cfg.c, cfg.k, cfg.W, cfg.sketch_seed)
    orc = Oracle(cfg.d, cfg.r, cfg.c, cfg.k, cfg.W, cfg.sketch_seed)
    st = wl.Structure(cfg, dev)
    v = wl.gradients(st, 0)
    if kind == "planted":
        v[:, st.planted_idx] *= 40.0
    if kind == "zero":
        v.zero_()
    u = torch.zeros_like(v)
    eng.bind(u, v, cfg.ncand)
    v_h = v.cpu().numpy()
    T, _ = orc.sketch_workers(v_h)
    Tf = T.astype(np.float32)
    out_idx = torch.empty(cfg.k, dtype=torch.int32, device=dev)
    out_val = torch.empty(cfg.k, device=dev)
    l2 = torch.zeros(1, dtype=torch.float64, device=dev)
    nheavy = torch.zeros(1, dtype=torch.int32, device=dev)
    for seed in (0, 12345678901234567):
        want = orc.heavymix(Tf, v_h, seed)
        eng.heavymix(torch.tensor(Tf, device=dev), seed, out_idx, out_val, l2, nheavy)
        assert eng.status() == S.OK
        assert abs(l2.item() - want["l2"]) <= 1e-12 * max(want["l2"], 1e-300)
        assert nheavy.item() == want["nheavy"]
        assert (out_idx.cpu().numpy() == want["out_idx"]).all()
        assert (out_val.cpu().numpy().view(np.uint32) == want["out_val"].view(np.uint32)).all()
    assert (v.cpu().numpy() == v_h).all()                 # the state is only read
    if kind == "planted":
        assert set(st.planted_idx.cpu().tolist()) <= set(want["out_idx"].tolist())
        assert 0 < want["nheavy"] <= cfg.k
    if kind == "zero":
        assert want["nheavy"] == cfg.d and want["out_idx"].tolist() == list(range(cfg.k))


def test_heavymix_on_the_step_table(cuda_device):
    """After ssgd_sketch_accumulate + merge on the GPU, HEAVYMIX on that table agrees with the oracle run
    on the same table."""
    dev = cuda_device
    cfg = wl.C1.scaled(d=300_000, c=8192, ncand=600, k=600)      # 292 planted coordinates, k well above them
    eng = S.Ssgd(cfg.d, cfg.r, cfg.c, cfg.k, cfg.W, cfg.sketch_seed)
    orc = Oracle(cfg.d, cfg.r, cfg.c, cfg.k, cfg.W, cfg.sketch_seed)
    u, v = wl.zero_state(cfg, dev)
    eng.bind(u, v, cfg.ncand)
    st = wl.Structure(cfg, dev)
    g = wl.gradients(st, 0)
    g[:, st.planted_idx] *= 40.0
    tables = torch.empty((cfg.W, cfg.r, cfg.c), device=dev)
    merged = torch.empty((cfg.r, cfg.c), device=dev)
    eng.sketch_accumulate(g, cfg.rho, tables)
    eng.sketch_merge(tables, merged)
    out_idx = torch.empty(cfg.k, dtype=torch.int32, device=dev)
    out_val = torch.empty(cfg.k, device=dev)
    nheavy = torch.zeros(1, dtype=torch.int32, device=dev)
    eng.heavymix(merged, 7, out_idx, out_val, None, nheavy)
    assert eng.status() == S.OK
    want = orc.heavymix(merged.cpu().numpy(), v.cpu().numpy(), 7)
    assert nheavy.item() == want["nheavy"]
    assert (out_idx.cpu().numpy() == want["out_idx"]).all()
    assert (out_val.cpu().numpy() == want["out_val"]).all()
    assert set(st.planted_idx.cpu().tolist()) <= set(want["out_idx"].tolist())


@pytest.mark.parametrize("d,k", [(200, 20), (200, 150), (100_003, 777), (100_003, 60_000)])
def test_heavymix_more_heavy_than_k_compares_full_magnitudes(cuda_device, d, k):
    """|H| > k (outside the paper's guarantee): one row, four buckets holding +-1.0 and +-(the next fp32 above
    1.0), so every coordinate is heavy and the magnitudes differ in the last mantissa bit only.  The k kept are
    the k largest under the full fp32 magnitude, ties to the smaller index -- the oracle's explicit branch."""
    dev = cuda_device
    one = np.float32(1.0)
    up = np.nextafter(one, np.float32(2.0))
    Tf = np.array([[one, up, -one, -up]], np.float32)
    eng = S.Ssgd(d, 1, 4, k, 2, 21)
    orc = Oracle(d, 1, 4, k, 2, 21)
    ld = (d + 3) // 4 * 4
    gen = torch.Generator(device=dev).manual_seed(d + k)
    v = torch.zeros((2, ld), device=dev)
    v[:, :d] = torch.randn((2, d), generator=gen, device=dev)
    u = torch.zeros_like(v)
    eng.bind(u, v, k)
    out_idx = torch.full((k,), -1, dtype=torch.int32, device=dev)
    out_val = torch.empty(k, device=dev)
    nheavy = torch.zeros(1, dtype=torch.int32, device=dev)
    v_h = v.cpu().numpy()
    for seed in (3, 4):
        want = orc.heavymix(Tf, v_h, seed)
        eng.heavymix(torch.tensor(Tf, device=dev), seed, out_idx, out_val, None, nheavy)
        assert eng.status() == S.OK
        assert nheavy.item() == want["nheavy"] == d
        assert (out_idx.cpu().numpy() == want["out_idx"]).all()
        assert (out_val.cpu().numpy().view(np.uint32) == want["out_val"].view(np.uint32)).all()
    assert want["out_idx"].tolist() != list(range(k))       # a key without the last mantissa bit would give this
    # the same context, a table with |H| <= k next: the gated second selection must stay out of the way
    Tf2 = np.array([[50.0, 0.25, -0.25, 0.125]], np.float32)
    want = orc.heavymix(Tf2, v_h, 9)
    if want["nheavy"] <= k:
        eng.heavymix(torch.tensor(Tf2, device=dev), 9, out_idx, out_val, None, nheavy)
        assert eng.status() == S.OK and nheavy.item() == want["nheavy"]
        assert (out_idx.cpu().numpy() == want["out_idx"]).all()
