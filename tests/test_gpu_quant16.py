"""16-bit sketches on the GPU: encodings and the merged table bit-exact against the oracle, and the effect
of the quantisation on what the step selects."""
import numpy as np
import pytest
import torch

from oracle import FMT_BF16, FMT_F16, Oracle, merge16, quantize16
from paper_1903_04488_b200 import ssgd as S
from paper_1903_04488_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("fmt", [FMT_F16, FMT_BF16])
def test_quantize_and_merge_bit_exact(cuda_device, fmt):
    dev = cuda_device
    cfg = wl.C2.scaled(d=50_000, W=5, c=1000, ncand=200, k=100)
    eng = S.Ssgd(cfg.d, cfg.r, cfg.c, cfg.k, cfg.W, 1)
    gen = torch.Generator(device=dev).manual_seed(3)
    scale = torch.pow(10.0, torch.randint(-9, 6, (cfg.W, cfg.r, cfg.c), generator=gen, device=dev).float())
    tables = torch.randn((cfg.W, cfg.r, cfg.c), generator=gen, device=dev) * scale
    tables[0, 0, :8] = torch.tensor([0.0, -0.0, 65504.0, 65519.0, 70000.0, -1e9, 5.9604645e-08, 2.9802322e-08], device=dev)
    q = torch.empty((cfg.W, cfg.r, cfg.c), dtype=torch.int16, device=dev)
    merged = torch.empty((cfg.r, cfg.c), device=dev)
    eng.sketch_quantize16(tables, fmt, q)
    eng.sketch_merge16(q, fmt, merged)
    torch.cuda.synchronize()
    q_o = quantize16(tables.cpu().numpy(), fmt)
    assert (q.cpu().numpy().view(np.uint16) == q_o).all()
    m_o = merge16(q_o, fmt)
    assert (merged.cpu().numpy().view(np.uint32) == m_o.view(np.uint32)).all()


@pytest.mark.parametrize("fmt", [FMT_F16, FMT_BF16])
def test_selection_survives_16_bit_sketches(cuda_device, fmt):
    """The faithful pipeline with the workers' sketches rounded to 16 bits picks nearly the same coordinates
    as with fp32 sketches (the paper reports no loss of accuracy from 16-bit sketches)."""
    dev = cuda_device
    cfg = wl.C2.scaled(d=1_000_003, W=8, c=32_768, ncand=10_000, k=5_000)
    g = wl.gradients(wl.Structure(cfg, dev), 0)

    def run(quantised):
        eng = S.Ssgd(cfg.d, cfg.r, cfg.c, cfg.k, cfg.W, cfg.sketch_seed)
        u, v = wl.zero_state(cfg, dev)
        eng.bind(u, v, cfg.ncand)
        tables = torch.empty((cfg.W, cfg.r, cfg.c), device=dev)
        merged = torch.empty((cfg.r, cfg.c), device=dev)
        eng.sketch_accumulate(g, cfg.rho, tables)
        if quantised:
            q = torch.empty(tables.shape, dtype=torch.int16, device=dev)
            eng.sketch_quantize16(tables, fmt, q)
            eng.sketch_merge16(q, fmt, merged)
        else:
            eng.sketch_merge(tables, merged)
        cand = torch.empty(cfg.ncand, dtype=torch.int32, device=dev)
        oi = torch.empty(cfg.k, dtype=torch.int32, device=dev)
        ov = torch.empty(cfg.k, device=dev)
        eng.unsketch_candidates(merged, cfg.ncand, cand)
        eng.exact_topk(cand, oi, ov)
        assert eng.status() == S.OK
        return cand.cpu().numpy(), oi.cpu().numpy()

    cand32, out32 = run(False)
    cand16, out16 = run(True)
    cand_overlap = np.intersect1d(cand32, cand16).size / cfg.ncand
    out_overlap = np.intersect1d(out32, out16).size / cfg.k
    print(f"fmt={fmt}: candidate overlap {cand_overlap:.4f}, final overlap {out_overlap:.4f}")
    assert cand_overlap > (0.97 if fmt == FMT_F16 else 0.90)
    assert out_overlap > (0.99 if fmt == FMT_F16 else 0.97)
