"""Parity at full size: the LLaMA-1B-shaped workload (1.14 B parameters, 146 blocks) in the launch configuration
``bench.py`` times (same tables, same tiles, the library's own budgeted assignment), and likewise the diffusion-UNet-
shaped (0.86 B parameters, per-level noise scales) and GPT-2-small-shaped (124 M parameters, Student-t gradients in the
embedding and attention blocks) workloads, checked on sampled outputs that the CPU oracle can compute one by one:

  * statistics of whole sampled blocks (a vector, a 4 M and a 16.7 M matrix), and the window values plus the
    anisotropy / signal-to-noise of the largest block (the 65.5 M-element token table);
  * after ten mixed steps, slices of element-wise blocks (fp32 Adam, RMS, SGD-m), whole quantisation blocks
    of 8-bit blocks, and whole factored blocks (their row/column statistics need every element).

Tolerances are the ones of test_gpu_parity.py.
"""
import numpy as np
import pytest
import torch

from oracle import baoc_oracle as O
from paper_2605_04711_b200 import workloads as W

pytestmark = pytest.mark.gpu

# Window lengths: the LLaMA-1B-shaped configuration states a 64-step window; the other two state none and take 8.
T_WINDOWS = {"llama_1b": 64, "unet": 8, "gpt2_small": 8}
N_STEPS = 10


def _ocfg(c):
    return O.Config(c.adaptive, c.momentum, c.decoupled_wd, c.factored, c.bits, lr=float(c.lr), beta1=float(c.beta1),
                    beta2=float(c.beta2), eps=float(c.eps), weight_decay=float(c.weight_decay),
                    quantizer="dynamic" if c.quantizer else "linear", af_beta2_schedule=bool(c.af_flags & 1),
                    af_clip=1.0 if c.af_flags & 2 else 0.0, af_relative_step=bool(c.af_flags & 4),
                    af_eps1=1e-30 if c.af_flags & 8 else 0.0)


def _close(got, ref):
    return abs(got - ref) <= 1e-4 * max(abs(ref), 1e-3)


def _slices(numel):
    """Three 8192-element windows (multiples of 256, so they hold whole quantisation blocks): start, middle, and
    the end of the block including its ragged tail."""
    if numel <= 3 * 8192:
        return [(0, numel)]
    mid = (numel // 2) // 256 * 256
    last = (numel - 8192 + 255) // 256 * 256
    return [(0, 8192), (mid, mid + 8192), (last, numel)]


CASES = {
    # workload: (parameter count or None, blocks with whole-block statistics, the largest block)
    "llama_1b": (1_139_345_408, ["l0.norm1", "l3.attn.k", "l5.ffn.up"], "tok_emb"),
    "unet": (None, ["in.b", "down1.attn0.self.q.w", "mid.attn.ff.gate.w"], "up3.res0.conv1.w"),
    "gpt2_small": (124_439_808, ["h0.ln1.w", "h3.attn.out.w", "h7.mlp.fc.w"], "tok_emb"),
}


@pytest.mark.parametrize("name", ["llama_1b", "unet", "gpt2_small"])
def test_sampled_parity_at_full_size(name):
    from paper_2605_04711_b200 import harness as H
    wl = W.make_workload(name, seed=0)
    numel, full_names, big_name = CASES[name]
    assert numel is None or wl.numel == numel
    if name == "unet":
        assert abs(wl.numel - 860e6) <= 0.02 * 860e6
    T_WINDOW = T_WINDOWS[name]
    assert name != "llama_1b" or T_WINDOW == wl.window
    sess = H.Session(wl, n_grad_sets=2)
    sess.init_params()
    o = O.Opts()
    name_to_i = {b.name: i for i, b in enumerate(wl.blocks)}
    full = [name_to_i[n] for n in full_names]                       # whole-block statistics
    big = name_to_i[big_name]                                       # the workload's largest block
    states = {i: O.stats_init(wl.blocks[i].numel) for i in full + [big]}
    for t in range(1, T_WINDOW + 1):
        k = sess.fill_grads(t)
        sess.sample_stats(k)
        for i, st in states.items():
            O.stats_step(st, sess.block_grad_host(k, i), o)
    run = sess.h.read_stats()
    for i, st in states.items():
        assert _close(run[i]["rho_bar"], st.rho_bar) and _close(run[i]["last_cos"], st.last_cos), wl.blocks[i].name
        assert run[i]["n_cos"] == T_WINDOW - 1
    # moments of the largest block on slices
    mv = [sess.h.view_tensor(big, w, torch.float32) for w in (0, 1)]
    for lo, hi in _slices(wl.blocks[big].numel):
        for dev, ref in ((mv[0], states[big].m), (mv[1], states[big].v)):
            got = dev[lo:hi].double().cpu().numpy()
            assert np.max(np.abs(got - ref[lo:hi])) <= 1e-6 * np.max(np.abs(ref))

    risk, st = sess.risk()
    for i in full:
        b = wl.blocks[i]
        raw = O.stats_finalize(states[i], sess.block_param_host(i), b.rows, b.cols, o)
        for key in ("A", "rho_bar", "snr", "C", "F", "Q32", "Q16", "Q8", "q10", "q90", "rho_mom",
                    "err_m8", "err_v8", "err_m16", "err_v16"):
            assert _close(st[i][key], raw[key]), (b.name, key, st[i][key], raw[key])
    # the largest block: exact quantiles (radix select across all of its tiles; 65.5 M elements for LLaMA-1B) and the SNR
    assert _close(st[big]["A"], O.anisotropy(states[big].v, o.eps)), (st[big]["A"],)
    assert _close(st[big]["snr"], O.snr(states[big].m, states[big].v, o.eps))
    del states, mv

    assign, obj, rc = sess.allocate(risk)
    assert rc == 0
    mem, _ = sess.h.cost_model()
    assert sum(int(mem[i, c]) for i, c in enumerate(assign)) <= int(wl.mem_budget_frac * 8 * wl.numel)
    cfgs = [_ocfg(c) for c in sess.configs]
    kinds = [O.config_kind(cfgs[c]) for c in assign]
    assert len(set(kinds)) >= 3, set(kinds)                         # the 25 % budget forces a mixed assignment
    sess.configure(assign)

    # sampled blocks per path: the first, the last and the largest block that took the path
    picks = []
    for kind in sorted(set(kinds)):
        ids = [i for i, k in enumerate(kinds) if k == kind]
        if kind == "F":
            ids = [i for i in ids if wl.blocks[i].numel <= 17_000_000] or ids
            chosen = {ids[0], ids[-1]}
        else:
            chosen = {ids[0], ids[-1], max(ids, key=lambda i: wl.blocks[i].numel)}
        picks += [(i, kind) for i in sorted(chosen)]
    samples = []
    for i, kind in picks:
        b = wl.blocks[i]
        for lo, hi in ([(0, b.numel)] if kind == "F" else _slices(b.numel)):
            n = hi - lo
            rows, cols = (b.rows, b.cols) if kind == "F" else (n, 1)
            samples.append(dict(i=i, kind=kind, lo=lo, hi=hi, rows=rows, cols=cols,
                                th=sess.param_views[i][lo:hi].double().cpu().numpy(),
                                st=O.step_init(cfgs[assign[i]], n, rows, cols)))
    for t in range(1, N_STEPS + 1):
        k = sess.fill_grads(T_WINDOW + t)
        sess.step(k, t)
        for s in samples:
            g = sess.grad_views[k][s["i"]][s["lo"]:s["hi"]].double().cpu().numpy()
            s["th"] = O.step(s["th"], g, s["st"], cfgs[assign[s["i"]]], s["rows"], s["cols"])
    torch.cuda.synchronize()
    cnt, _ = sess.h.nonfinite()
    assert cnt == 0
    bad_codes, n_codes = 0, 0
    for s in samples:
        i, lo, hi, ref = s["i"], s["lo"], s["hi"], s["st"]
        name = (wl.blocks[i].name, s["kind"], lo)
        got = sess.param_views[i][lo:hi].double().cpu().numpy()
        assert np.max(np.abs(got - s["th"])) <= 1e-6 * np.max(np.abs(s["th"])), name
        f32 = lambda w, a, b: sess.h.view_tensor(i, w, torch.float32)[a:b].double().cpu().numpy()
        rel = lambda x, y: float(np.max(np.abs(x - y)) / max(float(np.max(np.abs(y))), 1e-30))
        if s["kind"] == "A32":
            assert rel(f32(10, lo, hi), ref.m) <= 1e-6 and rel(f32(11, lo, hi), ref.v) <= 1e-6, name
        elif s["kind"] in ("R", "S"):
            assert rel(f32(10, lo, hi), ref.v if s["kind"] == "R" else ref.m) <= 1e-6, name
        elif s["kind"] == "F":
            assert rel(f32(10, 0, s["rows"]), ref.r) <= 1e-6 and rel(f32(11, 0, s["cols"]), ref.c) <= 1e-6, name
        elif s["kind"] == "A8":
            qm = sess.h.view_tensor(i, 10, torch.int8)[lo:hi].cpu().numpy().astype(np.int32)
            qv = sess.h.view_tensor(i, 11, torch.uint8)[lo:hi].cpu().numpy().astype(np.int32)
            dm, dv = np.abs(qm - ref.qm.astype(np.int32)), np.abs(qv - ref.qv.astype(np.int32))
            assert dm.max() <= 1 and dv.max() <= 1, name
            bad_codes += int((dm != 0).sum() + (dv != 0).sum())
            n_codes += 2 * qm.size
            q0, q1 = lo // 256, (hi + 255) // 256
            assert rel(f32(12, q0, q1), ref.am.astype(np.float64)) <= 1e-6, name
            assert rel(f32(13, q0, q1), ref.av.astype(np.float64)) <= 1e-6, name
    if n_codes:
        assert bad_codes <= 1e-4 * n_codes, (bad_codes, n_codes)


def test_one_block_beyond_two_to_the_31_elements():
    """Indexing past 32 bits: a single 32769 x 65537 block (2^31 + 98305 elements, odd row length, ragged tail; rows
    and columns are 32-bit in the ABI, their product is not) through the statistics pass and the fused step (SGD with
    momentum, so there is per-element state), checked on slices at the start, around element 2^31 and at the very
    end."""
    from paper_2605_04711_b200 import binding as B
    dev = torch.device("cuda:0")
    rows, cols = 32769, 65537
    n = rows * cols
    assert n > 2 ** 31
    cfgs = [B.make_config(0, 1, 1, 0, 32, lr=1e-2, beta1=0.9, weight_decay=0.01)]
    h = B.Baoc([(n, rows, cols)], cfgs)
    gen = torch.Generator(device=dev).manual_seed(5)
    theta = torch.empty(n, dtype=torch.float32, device=dev)
    grads = [torch.empty(n, dtype=torch.bfloat16, device=dev) for _ in range(2)]
    chunk = 2 ** 27
    for lo in range(0, n, chunk):                                      # chunked: no full-size fp32 temporaries
        hi = min(n, lo + chunk)
        theta[lo:hi] = 0.02 * torch.randn(hi - lo, generator=gen, device=dev)
        for g in grads:
            g[lo:hi] = (0.01 * torch.randn(hi - lo, generator=gen, device=dev)).to(torch.bfloat16)
    ws = torch.empty(h.stats_workspace_bytes(), dtype=torch.uint8, device=dev)
    h.bind_stats_workspace(ws)
    state = torch.empty(h.state_bytes([0]), dtype=torch.uint8, device=dev)
    h.configure([0], state)
    windows = [(0, 8192), (2 ** 31 - 4096, 2 ** 31 + 4096), (n - 5000, n)]
    th0 = [theta[a:b].double().cpu().numpy() for a, b in windows]
    o = O.Opts()
    for k in (0, 1):
        h.sample_stats([grads[k]])
        h.step([grads[k]], [theta], k + 1)
    torch.cuda.synchronize()
    run = h.read_stats()[0]
    # the cosine of the two gradients over all 2^31 + 4100 elements, from chunked double-precision dot products
    dot = n1 = n2 = 0.0
    for lo in range(0, n, chunk):
        a, b = grads[0][lo:lo + chunk].double(), grads[1][lo:lo + chunk].double()
        dot += float(a @ b); n1 += float(a @ a); n2 += float(b @ b)
    want = dot / (np.sqrt(n1) * np.sqrt(n2) + o.eps)
    assert abs(run["last_cos"] - want) <= 1e-4 * max(abs(want), 1e-3) and run["n_cos"] == 1
    c = O.Config(0, 1, 1, 0, 32, lr=float(cfgs[0].lr), beta1=float(cfgs[0].beta1), weight_decay=float(cfgs[0].weight_decay))
    m_dev = h.view_tensor(0, 10, torch.float32)
    mhat = h.view_tensor(0, 0, torch.float32)
    for (a, b), t0 in zip(windows, th0):
        st, ss, th = O.step_init(c, b - a, b - a, 1), O.stats_init(b - a), t0
        for k in (0, 1):
            g = grads[k][a:b].double().cpu().numpy()
            O.stats_step(ss, g, o)
            th = O.step(th, g, st, c, b - a, 1)
        got = theta[a:b].double().cpu().numpy()
        assert np.max(np.abs(got - th)) <= 1e-6 * np.max(np.abs(th)), (a, b)
        assert np.max(np.abs(m_dev[a:b].double().cpu().numpy() - st.m)) <= 1e-6 * np.max(np.abs(st.m))
        assert np.max(np.abs(mhat[a:b].double().cpu().numpy() - ss.m)) <= 1e-6 * np.max(np.abs(ss.m))


def test_every_tuple_family_in_one_step_at_full_size():
    """All fifteen instantiable tuples (the two alternative readings included) dealt round-robin over the blocks of the LLaMA-1B-shaped workload, so that one
    step launches every kernel instance (headline paths, stateless / bf16 dense paths, 8-bit single-moment paths) over
    its stretch of the tile table; ten steps, checked on slices (whole blocks for the factored ones)."""
    from paper_2605_04711_b200 import binding as B, harness as H
    wl = W.make_workload("llama_1b", seed=1)
    bcfgs = B.extended_configs()
    sess = H.Session(wl, configs=bcfgs, n_grad_sets=2)
    sess.init_params()
    cfgs = [_ocfg(c) for c in bcfgs]
    factored = {3: 2, 11: 7, 12: 9, 14: 2}                           # vectors take RMS scaling at the same precision
    assign = []
    for i, b in enumerate(wl.blocks):
        c = i % len(bcfgs)
        assign.append(factored[c] if (c in factored and b.cols <= 1) else c)
    kinds = [O.config_kind(cfgs[c]) for c in assign]
    assert set(kinds) == {"A32", "A8", "R", "F", "S", "G", "A16", "R16", "S16", "R8", "S8", "F16", "F8", "A8N"}
    assert any(cfgs[c].af_clip for c in assign)                      # the factored tuple with Adafactor's options is among them
    sess.configure(assign)
    mem, _ = sess.h.cost_model()
    assert sess.h.query().state_bytes == sum(int(mem[i, c]) for i, c in enumerate(assign))
    picks = []
    for kind in sorted(set(kinds)):
        ids = [i for i, k in enumerate(kinds) if k == kind]
        if kind.startswith("F"):
            ids = [i for i in ids if wl.blocks[i].numel <= 17_000_000] or ids
            picks += [(ids[0], kind)]
            with_options = [i for i in ids if cfgs[assign[i]].af_clip and i != ids[0]]
            picks += [(with_options[0], kind)] if with_options else []
        else:
            picks += [(i, kind) for i in sorted({ids[0], max(ids, key=lambda i: wl.blocks[i].numel)})]
    samples = []
    for i, kind in picks:
        b = wl.blocks[i]
        whole = kind.startswith("F")
        for lo, hi in ([(0, b.numel)] if whole else _slices(b.numel)):
            n = hi - lo
            rows, cols = (b.rows, b.cols) if whole else (n, 1)
            samples.append(dict(i=i, kind=kind, lo=lo, hi=hi, rows=rows, cols=cols,
                                th=sess.param_views[i][lo:hi].double().cpu().numpy(),
                                st=O.step_init(cfgs[assign[i]], n, rows, cols)))
    launches0 = sess.h.query().kernel_launches
    for t in range(1, N_STEPS + 1):
        k = sess.fill_grads(t)
        sess.step(k, t)
        for s in samples:
            g = sess.grad_views[k][s["i"]][s["lo"]:s["hi"]].double().cpu().numpy()
            s["th"] = O.step(s["th"], g, s["st"], cfgs[assign[s["i"]]], s["rows"], s["cols"])
    torch.cuda.synchronize()
    assert sess.h.query().kernel_launches - launches0 == N_STEPS * 7    # row/column reduce + combine, two norms kernels, three instances
    assert sess.h.nonfinite()[0] == 0
    bad, total = 0, 0
    rel = lambda x, y: float(np.max(np.abs(x - y)) / max(float(np.max(np.abs(y))), 1e-30))
    for s in samples:
        i, lo, hi, ref, kind = s["i"], s["lo"], s["hi"], s["st"], s["kind"]
        name = (wl.blocks[i].name, kind, lo)
        got = sess.param_views[i][lo:hi].double().cpu().numpy()
        assert np.max(np.abs(got - s["th"])) <= 1e-6 * np.max(np.abs(s["th"])), name
        view = lambda w, dt, a, b: sess.h.view_tensor(i, w, dt)[a:b]
        f32 = lambda w, a, b: view(w, torch.float32, a, b).double().cpu().numpy()
        bits = lambda w, a, b: view(w, torch.bfloat16, a, b).view(torch.int16).cpu().numpy().astype(np.int32)
        want_bits = lambda x: torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().astype(np.int32)
        q0, q1 = lo // 256, (hi + 255) // 256

        def codes(w, dt, ref_q, a=lo, b=hi):
            nonlocal bad, total
            d = np.abs(view(w, dt, a, b).cpu().numpy().astype(np.int32) - ref_q.astype(np.int32))
            assert d.max() <= 1, name
            bad += int((d != 0).sum()); total += d.size

        def patterns(w, ref_x, a=lo, b=hi):
            nonlocal bad, total
            d = np.abs(bits(w, a, b) - want_bits(ref_x))
            assert d.max() <= 1, name
            bad += int((d != 0).sum()); total += d.size

        if kind == "A32":
            assert rel(f32(10, lo, hi), ref.m) <= 1e-6 and rel(f32(11, lo, hi), ref.v) <= 1e-6, name
        elif kind in ("R", "S"):
            assert rel(f32(10, lo, hi), ref.v if kind == "R" else ref.m) <= 1e-6, name
        elif kind == "F":
            assert rel(f32(10, 0, s["rows"]), ref.r) <= 1e-6 and rel(f32(11, 0, s["cols"]), ref.c) <= 1e-6, name
        elif kind == "F16":
            patterns(10, ref.r, 0, s["rows"]); patterns(11, ref.c, 0, s["cols"])
        elif kind == "F8":
            codes(10, torch.uint8, ref.qr, 0, s["rows"]); codes(11, torch.uint8, ref.qc, 0, s["cols"])
            assert rel(f32(12, 0, len(ref.ar)), ref.ar.astype(np.float64)) <= 1e-6, name
            assert rel(f32(13, 0, len(ref.ac)), ref.ac.astype(np.float64)) <= 1e-6, name
        elif kind == "A16":
            patterns(10, ref.m); patterns(11, ref.v)
        elif kind in ("R16", "S16"):
            patterns(10, ref.v if kind == "R16" else ref.m)
        elif kind == "A8N":
            codes(10, torch.uint8, ref.qm); codes(11, torch.uint8, ref.qv)
            assert rel(f32(12, q0, q1), ref.am.astype(np.float64)) <= 1e-6, name
            assert rel(f32(13, q0, q1), ref.av.astype(np.float64)) <= 1e-6, name
        elif kind == "A8":
            codes(10, torch.int8, ref.qm); codes(11, torch.uint8, ref.qv)
            assert rel(f32(12, q0, q1), ref.am.astype(np.float64)) <= 1e-6, name
            assert rel(f32(13, q0, q1), ref.av.astype(np.float64)) <= 1e-6, name
        elif kind in ("R8", "S8"):
            codes(10, torch.uint8 if kind == "R8" else torch.int8, ref.qv if kind == "R8" else ref.qm)
            assert rel(f32(11, q0, q1), (ref.av if kind == "R8" else ref.am).astype(np.float64)) <= 1e-6, name
    assert total > 0 and bad <= 1e-4 * total, (bad, total)
