"""The allocation-free statistics call against the handle-based one.

Some callers cannot allocate device memory when they need a block's statistics (allocator hooks, out-of-memory
callbacks, trainers whose caching allocator must not fall through to cudaMalloc), so the library offers
``baoc_sample_stats_noalloc``, whose scratch is a fixed array inside the library.  This file checks, through
the C ABI, that it gives what ``baoc_sample_stats`` gives on the same data, on two calls in a row (the second
call finds the first call's leftovers in the shared scratch).  It is collected last on purpose: a run that
stops at the first failure has then already run every other test.
"""
import numpy as np
import pytest
import torch

from paper_2605_04711_b200 import workloads as W

pytestmark = pytest.mark.gpu


def test_noalloc_matches_the_handle_path_on_two_calls_in_a_row():
    from paper_2605_04711_b200 import binding as B
    from paper_2605_04711_b200 import harness as H

    # one matrix block that spans several tiles with a ragged tail, and one short vector
    blocks = [W.Block("mat", 333, 77, stability=0.6, tau=1.0, scale=2e-2), W.Block("vec", 5, 1, stability=0.3, tau=0.5)]
    wl = W.Workload("noalloc", blocks, window=3, mem_budget_frac=0.5, time_budget=1.3, seed=17)
    sess = H.Session(wl, n_grad_sets=1)
    dev = sess.device
    mine = []
    for b in blocks:
        mine.append(dict(gprev=torch.zeros(b.numel, dtype=torch.bfloat16, device=dev),
                         m=torch.zeros(b.numel, dtype=torch.float32, device=dev),
                         v=torch.zeros(b.numel, dtype=torch.float32, device=dev),
                         out=torch.full((4,), -7.0, dtype=torch.float64, device=dev)))
    m_prev = [np.zeros(b.numel) for b in blocks]
    for t in (1, 2, 3):
        sess.fill_grads(t)
        sess.sample_stats(0)
        ref = sess.h.read_stats()
        for i, b in enumerate(blocks):
            s = mine[i]
            B.sample_stats_noalloc(sess.grad_views[0][i], s["gprev"], s["m"], s["v"], s["out"])
        torch.cuda.synchronize()
        for i, b in enumerate(blocks):
            s = mine[i]
            out = s["out"].cpu().numpy()
            want_cos = ref[i]["last_cos"] if t > 1 else 0.0
            assert abs(out[0] - want_cos) <= 1e-4 * max(abs(want_cos), 1e-3), (t, b.name, out[0], want_cos)
            g = sess.block_grad_host(0, i)
            assert abs(out[1] - float(np.dot(g, g))) <= 1e-4 * float(np.dot(g, g))
            # the cosine with the first moment before the update, and that moment's squared norm
            m_before = m_prev[i]
            want_m2 = float(np.dot(m_before, m_before))
            assert abs(out[3] - want_m2) <= 1e-4 * max(want_m2, 1e-30), (t, b.name, out[3], want_m2)
            if t == 2:                                              # the handle's running value starts at its first cosine
                assert abs(out[2] - ref[i]["rho_mom"]) <= 1e-4 * max(abs(ref[i]["rho_mom"]), 1e-3), (b.name, out[2])
            elif t == 1:
                assert out[2] == 0.0 and out[3] == 0.0              # zero moment: the cosine is not a number, counted as 0
            for which, key, dt in ((0, "m", torch.float32), (1, "v", torch.float32), (2, "gprev", torch.bfloat16)):
                want = sess.h.view_tensor(i, which, dt)
                assert torch.equal(s[key], want), (t, b.name, key)
            m_prev[i] = s["m"].double().cpu().numpy()


@pytest.mark.parametrize("numel", [2 * 1024 * 1024 + 4099, None])
def test_noalloc_at_size(numel):
    """A block with more tiles than the combine kernel has threads and a ragged tail (2 Mi + 4099 elements: 514
    tiles), and a block of exactly the documented maximum (64 Mi elements: every slot of the built-in scratch in
    use), each against the handle-based path on two observations in a row."""
    from paper_2605_04711_b200 import binding as B
    dev = torch.device("cuda:0")
    n = B.NOALLOC_MAX_NUMEL if numel is None else numel
    gen = torch.Generator(device=dev).manual_seed(29)
    h = B.Baoc([(n, n, 1)], B.default_configs())
    ws = torch.empty(h.stats_workspace_bytes(), dtype=torch.uint8, device=dev)
    h.bind_stats_workspace(ws)
    gprev = torch.zeros(n, dtype=torch.bfloat16, device=dev)
    m = torch.zeros(n, dtype=torch.float32, device=dev)
    v = torch.zeros(n, dtype=torch.float32, device=dev)
    out = torch.full((4,), -7.0, dtype=torch.float64, device=dev)
    base = torch.randn(n, generator=gen, device=dev)
    for t in (1, 2):
        g = (0.01 * (base + 0.5 * torch.randn(n, generator=gen, device=dev))).to(torch.bfloat16)
        h.sample_stats([g])
        B.sample_stats_noalloc(g, gprev, m, v, out)
        torch.cuda.synchronize()
        ref = h.read_stats()[0]
        o4 = out.cpu().numpy()
        want_cos = ref["last_cos"] if t > 1 else 0.0
        assert abs(o4[0] - want_cos) <= 1e-4 * max(abs(want_cos), 1e-3), (t, o4[0], want_cos)
        n2 = float((g.double() ** 2).sum())
        assert abs(o4[1] - n2) <= 1e-4 * n2
        if t == 2:
            assert 0.3 < o4[0] < 1.0
            assert abs(o4[2] - ref["rho_mom"]) <= 1e-4 * max(abs(ref["rho_mom"]), 1e-3)
        for which, mine, dt in ((0, m, torch.float32), (1, v, torch.float32), (2, gprev, torch.bfloat16)):
            assert torch.equal(mine, h.view_tensor(0, which, dt)), (t, which)


def test_noalloc_rejects_oversized_and_misaligned_input():
    from paper_2605_04711_b200 import binding as B
    dev = torch.device("cuda:0")
    g = torch.zeros(64, dtype=torch.bfloat16, device=dev)
    m = torch.zeros(64, dtype=torch.float32, device=dev)
    out = torch.zeros(4, dtype=torch.float64, device=dev)
    with pytest.raises(B.BaocError) as e:
        B.sample_stats_noalloc(g, g.clone(), m, m.clone(), out, numel=B.NOALLOC_MAX_NUMEL + 1)
    assert e.value.code == B.E_WORKSPACE and "BAOC_NOALLOC_MAX_NUMEL" in str(e.value)
    with pytest.raises(B.BaocError) as e:
        B.sample_stats_noalloc(g[1:33], g.clone(), m, m.clone(), out, numel=32)
    assert e.value.code == B.E_ALIGN
