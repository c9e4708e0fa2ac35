"""Checkpoint / resume of the method's state (u, v per worker; Algorithm 3 line 1) and the lifecycle rules of
the deferred zero-out (Algorithm 3 line 13 kept as marks in the workspace until the next step or ssgd_flush).

Integer-valued gradients and rho = 1/2 make every operation exact, the reductions into the sketch included, so
two runs that see the same state produce the same bits whatever order the reductions take."""
import io

import numpy as np
import pytest
import torch

from oracle import Oracle
from paper_1903_04488_b200 import ssgd as S
from paper_1903_04488_b200 import workloads as wl

pytestmark = pytest.mark.gpu

CFG = wl.C2.scaled(d=120_003, W=3, c=2048, ncand=2400, k=900)
RHO = 0.5


def int_gradients(step, dev):
    gen = torch.Generator(device=dev).manual_seed(4242 + step)
    g = torch.zeros((CFG.W, CFG.ld), device=dev)
    g[:, :CFG.d] = torch.randint(-40, 41, (CFG.W, CFG.d), generator=gen, device=dev).float()
    heavy = torch.arange(17, CFG.d, 97, device=dev)[: 2 * CFG.k]
    g[:, heavy] += 64.0 * (1 + (heavy % 5)).float()          # coordinates worth choosing, the same for every worker
    return g


def fresh(dev, zero_mode):
    eng = S.Ssgd(CFG.d, CFG.r, CFG.c, CFG.k, CFG.W, CFG.sketch_seed)
    u, v = wl.zero_state(CFG, dev)
    eng.bind(u, v, CFG.ncand)
    eng.set_zero_mode(zero_mode)
    return eng, u, v


def run(eng, dev, steps):
    out = []
    oi = torch.empty(CFG.k, dtype=torch.int32, device=dev)
    ov = torch.empty(CFG.k, device=dev)
    for t in steps:
        eng.step(int_gradients(t, dev), RHO, CFG.ncand, oi, ov)
        assert eng.status() == S.OK
        out.append((oi.cpu().numpy().copy(), ov.cpu().numpy().copy()))
    return out


@pytest.mark.parametrize("zero_mode", [S.ZERO_DEFERRED, S.ZERO_EAGER])
def test_ten_steps_equal_five_plus_checkpoint_plus_five(cuda_device, zero_mode):
    dev = cuda_device
    eng_a, u_a, v_a = fresh(dev, zero_mode)
    want = run(eng_a, dev, range(10))
    eng_a.flush()

    eng_b, u_b, v_b = fresh(dev, zero_mode)
    got = run(eng_b, dev, range(5))
    eng_b.flush()                                           # the checkpoint rule: flush, then save u and v
    buf = io.BytesIO()
    torch.save({"u": u_b.cpu(), "v": v_b.cpu()}, buf)
    del eng_b, u_b, v_b
    buf.seek(0)
    ck = torch.load(buf)
    eng_c = S.Ssgd(CFG.d, CFG.r, CFG.c, CFG.k, CFG.W, CFG.sketch_seed)   # hashes are a function of the seed
    u_c, v_c = ck["u"].to(dev), ck["v"].to(dev)
    eng_c.bind(u_c, v_c, CFG.ncand)
    eng_c.set_zero_mode(zero_mode)
    got += run(eng_c, dev, range(5, 10))
    eng_c.flush()
    for t, ((wi, wv), (gi, gv)) in enumerate(zip(want, got)):
        assert (wi == gi).all(), f"step {t}: chosen coordinates differ after the resume"
        assert (wv.view(np.uint32) == gv.view(np.uint32)).all(), f"step {t}: values differ after the resume"
    assert torch.equal(u_a, u_c) and torch.equal(v_a, v_c)
    # and the whole sequence is what the oracle computes (every operation is exact on these inputs)
    orc = Oracle(CFG.d, CFG.r, CFG.c, CFG.k, CFG.W, CFG.sketch_seed)
    u_o = np.zeros((CFG.W, CFG.ld), np.float32)
    v_o = np.zeros_like(u_o)
    for t in range(10):
        o = orc.step(int_gradients(t, dev).cpu().numpy(), RHO, u_o, v_o, CFG.ncand)
        order = np.argsort(o["out_idx"])
        assert (o["out_idx"][order] == want[t][0]).all() and (o["out_val"][order] == want[t][1]).all()
    assert (u_a.cpu().numpy() == u_o).all() and (v_a.cpu().numpy() == v_o).all()


def test_saving_without_the_flush_loses_line_13_and_the_library_says_so(cuda_device):
    """With the zero-out deferred, u and v in memory still hold the chosen coordinates' values after a step: a
    checkpoint taken then differs from the real state, and the context refuses to be rebound or destroyed until
    the marks are applied (ssgd_flush) or given up on purpose (ssgd_unbind)."""
    dev = cuda_device
    lib = S.lib()
    eng, u, v = fresh(dev, S.ZERO_DEFERRED)
    (idx, _), = run(eng, dev, [0])
    chosen = torch.tensor(idx, device=dev).long()
    assert (v[:, chosen] != 0).any()                        # memory is not the state yet
    u2, v2 = wl.zero_state(CFG, dev)
    ws2 = torch.empty(eng.workspace_bytes(CFG.ncand), dtype=torch.uint8, device=dev)
    with pytest.raises(S.SsgdError) as e:
        eng.bind(u2, v2, CFG.ncand, ws2)
    assert e.value.code == S.EPENDING
    assert lib.ssgd_destroy(eng._h) == S.EPENDING           # still alive and usable:
    assert b"ssgd_flush" in lib.ssgd_strerror(S.EPENDING)
    eng.flush()
    assert (v[:, chosen] == 0).all() and (u[:, chosen] == 0).all()
    eng.bind(u2, v2, CFG.ncand, ws2)                        # accepted now
    # the explicit way out: unbind discards the marks, the old buffers keep their values
    (idx, _), = run(eng, dev, [1])
    chosen = torch.tensor(idx, device=dev).long()
    before = v2.clone()
    eng.unbind()
    torch.cuda.synchronize()
    assert torch.equal(v2, before) and (v2[:, chosen] != 0).any()
    with pytest.raises(S.SsgdError) as e:
        eng.flush()
    assert e.value.code == S.ENOTBOUND
    eng.bind(u, v, CFG.ncand)
    # eager mode never has anything pending
    eng.set_zero_mode(S.ZERO_EAGER)
    run(eng, dev, [2])
    eng.bind(u2, v2, CFG.ncand, ws2)
