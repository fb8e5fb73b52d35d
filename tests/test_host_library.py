"""Host side of the C ABI, no GPU: defaults, argument checks, call order, cost
model, normalisation and risk against the oracle, and the exact allocator
against brute force."""
import math

import numpy as np
import pytest

from oracle import baoc_oracle as O
from paper_2605_04711_b200 import workloads as W


@pytest.fixture(scope="module")
def B():
    from paper_2605_04711_b200 import build
    build.build()
    from paper_2605_04711_b200 import binding
    return binding


def _ocfg(c):
    """Oracle view of a library configuration (fp32 hyper-parameters widened exactly)."""
    return O.Config(c.adaptive, c.momentum, c.decoupled_wd, c.factored, c.bits, lr=float(c.lr), beta1=float(c.beta1),
                    beta2=float(c.beta2), eps=float(c.eps), weight_decay=float(c.weight_decay))


def test_default_opts_match_oracle_defaults(B):
    o, ref = B.default_opts(), O.Opts()
    for k in ("beta_m", "beta_v", "beta_rho", "eps", "a_lo", "a_hi", "rho_lo", "rho_hi", "snr_lo", "snr_hi", "gamma",
              "eps_adam"):
        assert getattr(o, k) == getattr(ref, k), k
    assert tuple(o.w) == ref.w and o.use_snr == 1 and o.qblock == 256


def test_create_rejects_bad_arguments(B):
    cfgs = B.default_configs()
    with pytest.raises(B.BaocError):
        B.Baoc([(10, 5, 3)], cfgs)                       # rows*cols != numel
    with pytest.raises(B.BaocError):
        B.Baoc([(0, 0, 1)], cfgs)
    with pytest.raises(B.BaocError):
        B.Baoc([(16, 16, 1)], [B.make_config(1, 1, 1, 0, 4)])   # bits
    o = B.default_opts(); o.qblock = 128
    with pytest.raises(B.BaocError):
        B.Baoc([(16, 16, 1)], cfgs, o)
    with pytest.raises(B.BaocError):
        B.Baoc([(16, 16, 1)], cfgs * 7)                   # more than 32 configurations


def test_call_order_is_enforced_without_touching_a_gpu(B):
    h = B.Baoc([(512, 512, 1), (64 * 64, 64, 64)], B.default_configs())
    tab = (B.C.c_void_p * 2)(16, 32)
    for fn in (lambda: h.sample_stats(tab), lambda: h.risk(tab), lambda: h.read_stats()):
        with pytest.raises(B.BaocError) as e:
            fn()
        assert e.value.code == B.E_STATE
    with pytest.raises(B.BaocError) as e:
        h.step(tab, tab, 1)
    assert e.value.code == B.E_STATE
    with pytest.raises(B.BaocError) as e:
        h.state_bytes([0, 7])
    assert e.value.code == B.E_INVALID
    with pytest.raises(B.BaocError) as e:
        h.state_bytes([3, 0])                             # factored on a vector block
    assert e.value.code == B.E_INVALID
    assert h.state_bytes([0, 3]) > 0
    info = h.query()
    assert (info.n_blocks, info.n_cfg, info.numel, info.kernel_launches) == (2, 5, 512 + 4096, 0)
    assert info.stats_bytes_per_call == 22 * (512 + 4096)
    assert h.stats_workspace_bytes() > 10 * (512 + 4096)


def test_cost_model_matches_oracle_state_bytes(B):
    wl = W.make_workload("resnet50")
    cfgs = B.default_configs() + [B.make_config(1, 1, 1, 0, 16), B.make_config(0, 1, 0, 0, 8)]
    h = B.Baoc(wl.blocks, cfgs)
    mem, ratio = h.cost_model()
    for i, b in enumerate(wl.blocks):
        for c, k in enumerate(cfgs):
            assert mem[i, c] == O.state_bytes(_ocfg(k), b.numel, b.rows, b.cols)
    d = wl.blocks[0].numel
    assert ratio[0, 0] == 1.0 and abs(ratio[0, 2] - 18.0 / 26.0) < 1e-12 and abs(ratio[0, 4] - 18.0 / 26.0) < 1e-12
    assert abs(ratio[0, 1] - (10 * d + 2 * mem[0, 1]) / (26.0 * d)) < 1e-12


def test_risk_from_raw_matches_oracle(B):
    rng = np.random.default_rng(3)
    n = 40
    cfgs = B.default_configs() + [B.make_config(1, 1, 0, 0, 16), B.make_config(0, 0, 0, 1, 8)]
    o = B.default_opts()
    o.w[0], o.w[1], o.w[2], o.w[3], o.w[4] = 1.5, 0.5, 2.0, 1.0, 3.0
    h = B.Baoc([(64, 8, 8)] * n, cfgs, o)
    raw = []
    for i in range(n):
        raw.append(dict(A=rng.uniform(-1, 4), rho_bar=rng.uniform(-1, 1), snr=rng.uniform(0, 20), C=rng.uniform(0, 5),
                        F=rng.uniform(0, 1.5), Q32=1.0, Q16=rng.uniform(0.9, 1.0), Q8=rng.uniform(-0.2, 1.0)))
    raw[0].update(A=math.log(2.0), rho_bar=0.4, snr=math.e - 1.0)
    risk, st = h.risk_from_raw(raw)
    oo = O.Opts(w=(1.5, 0.5, 2.0, 1.0, 3.0))
    for i in range(n):
        z = O.normalise(raw[i], oo)
        for k in ("s_A", "s_rho", "s_snr", "s_M", "C_tilde", "s_F", "lQ32", "lQ16", "lQ8"):
            assert st[i][k] == pytest.approx(z[k], rel=1e-14, abs=1e-15), k
        for c, k in enumerate(cfgs):
            assert risk[i, c] == pytest.approx(O.risk(z, _ocfg(k), oo), rel=1e-13, abs=1e-15)
    assert st[0]["s_A"] == 0.0 and abs(st[0]["s_M"] - 0.25) < 1e-15
    o2 = B.default_opts(); o2.use_snr = 0
    _, st2 = B.Baoc([(64, 8, 8)] * n, cfgs, o2).risk_from_raw(raw)
    assert abs(st2[0]["s_M"] - 0.5) < 1e-15


def _brute(B, cfgs, blocks, risk, mem, ratio, b_mem, b_time, forbid=None, pref=None):
    oo = O.Opts()
    n, K = risk.shape
    oc = [_ocfg(c) for c in cfgs]
    phi = [[O.phi_fixed(O.objective(risk[i, c], oc[c], oo, 0.0 if pref is None else pref[i, c])) for c in range(K)]
           for i in range(n)]
    rfx = [[O.ratio_fixed(ratio[i, c]) for c in range(K)] for i in range(n)]
    fb = np.zeros((n, K), np.uint8) if forbid is None else forbid.copy()
    for i, b in enumerate(blocks):
        for c, k in enumerate(oc):
            kind = O.config_kind(k)
            if kind == "unsupported" or (kind == "F" and b[2] <= 1):
                fb[i, c] = 1
    return O.allocate_bruteforce(phi, mem.tolist(), rfx, b_mem, O.time_cap_fixed(n, b_time), fb.tolist())


@pytest.mark.parametrize("seed", range(6))
def test_allocator_equals_brute_force(B, seed):
    rng = np.random.default_rng(seed)
    cfgs = B.default_configs() + [B.make_config(0, 0, 1, 0, 32)]      # last one cannot be instantiated
    K = len(cfgs)
    for trial in range(60):
        n = int(rng.integers(1, 8))
        blocks = [(64, 8, 8) if rng.random() < 0.6 else (64, 64, 1) for _ in range(n)]
        h = B.Baoc(blocks, cfgs)
        if trial % 2 == 0:                                           # small integers: many exact ties
            risk = rng.integers(0, 4, (n, K)).astype(np.float64) / 4
            mem = rng.integers(1, 5, (n, K)).astype(np.int64)
            ratio = rng.integers(1, 4, (n, K)).astype(np.float64) / 2
        else:
            risk = rng.random((n, K)) * 3
            mem = rng.integers(1, 100000, (n, K)).astype(np.int64)
            ratio = rng.random((n, K)) * 2
        b_mem = max(0, int(mem.min(axis=1).sum() + rng.integers(0, int(mem.max()) * n // 2 + 1)) - int(trial % 7 == 0) * 3)
        b_time = float(rng.choice([0.6, 1.0, 1.3, 5.0]))
        forbid = (rng.random((n, K)) < 0.15).astype(np.uint8) if trial % 3 == 0 else None
        pref = (rng.random((n, K)) < 0.2) * 0.25 if trial % 4 == 0 else None
        want, want_val = _brute(B, cfgs, blocks, risk, mem, ratio, b_mem, b_time, forbid, pref)
        if want is None:
            with pytest.raises(B.BaocError) as e:
                h.allocate(risk, mem, ratio, b_mem, b_time, forbid, pref)
            assert e.value.code == B.E_INFEASIBLE
            continue
        asg, obj, rc = h.allocate(risk, mem, ratio, b_mem, b_time, forbid, pref)
        assert rc == 0
        assert asg.tolist() == want                                   # bit-exact, tie-break included
        assert obj == want_val / 2.0 ** 30
        assert sum(mem[i, c] for i, c in enumerate(asg)) <= b_mem


def test_allocator_properties_on_a_large_problem(B):
    wl = W.make_workload("llama_1b")
    cfgs = B.default_configs()
    h = B.Baoc(wl.blocks, cfgs)
    mem, ratio = h.cost_model()
    rng = np.random.default_rng(0)
    n = len(wl.blocks)
    base = np.array([0.0, 0.05, 0.4, 0.8, 0.9])
    risk = base[None, :] * rng.uniform(0.2, 1.8, (n, 5))
    full = 8 * wl.numel
    prev_obj, prev_mem = None, None
    for frac in (0.25, 0.3, 0.5, 1.0):
        asg, obj, rc = h.allocate(risk, mem, ratio, int(frac * full), 1.3)
        assert rc == 0
        used = sum(int(mem[i, c]) for i, c in enumerate(asg))
        assert used <= int(frac * full)
        for i, c in enumerate(asg):
            assert not (c == 3 and wl.blocks[i].cols <= 1)            # factored never lands on a vector
        if prev_obj is not None:
            assert obj <= prev_obj + 1e-12 and used >= prev_mem       # more budget: never worse, never less memory here
        prev_obj, prev_mem = obj, used
    assert asg.tolist() == [0] * n                                    # whole budget and zero risk for fp32 Adam
    with pytest.raises(B.BaocError) as e:
        h.allocate(risk, mem, ratio, 1000, 1.3)
    assert e.value.code == B.E_INFEASIBLE
    # a time budget below every ratio is infeasible as well
    with pytest.raises(B.BaocError) as e:
        h.allocate(risk, mem, ratio, full, 0.1)
    assert e.value.code == B.E_INFEASIBLE


def test_allocator_time_budget_binds_and_node_limit_warns(B):
    wl = W.make_workload("resnet50")
    cfgs = B.default_configs()
    h = B.Baoc(wl.blocks, cfgs)
    mem, _ = h.cost_model()
    ratio = W.time_ratio_table(wl, [1.0, 1.25, 0.8, 1.5, 0.7]).numpy()
    rng = np.random.default_rng(1)
    risk = rng.random((len(wl.blocks), 5))
    asg, obj, rc = h.allocate(risk, mem, ratio, int(0.4 * 8 * wl.numel), 1.1)
    assert rc == 0
    assert sum(ratio[i, c] for i, c in enumerate(asg)) / len(asg) <= 1.1 + 1e-6
    asg2, obj2, _ = h.allocate(risk, mem, ratio, int(0.4 * 8 * wl.numel), 0.95)
    assert obj2 >= obj and sum(ratio[i, c] for i, c in enumerate(asg2)) / len(asg2) <= 0.95 + 1e-6
    o = B.default_opts(); o.node_limit = 170
    h3 = B.Baoc(wl.blocks, cfgs, o)
    asg3, obj3, rc3 = h3.allocate(risk, mem, ratio, int(0.4 * 8 * wl.numel), 1.1)
    if rc3 == B.W_NODE_LIMIT:
        assert sum(int(mem[i, c]) for i, c in enumerate(asg3)) <= int(0.4 * 8 * wl.numel)
        assert obj3 >= obj - 1e-12


def test_export_import_blob_without_device_state(B):
    blocks = [(64, 8, 8), (5, 5, 1)]
    h = B.Baoc(blocks, B.default_configs())
    blob = h.export_state()
    assert len(blob) >= 40
    B.Baoc(blocks, B.default_configs()).import_state(blob)                     # nothing bound, nothing configured: fine
    other_lr = B.default_configs()
    other_lr[0].lr = 5e-4
    B.Baoc(blocks, other_lr).import_state(blob)                                # hyper-parameters may differ on resume
    for bad_handle in (B.Baoc([(64, 8, 8), (6, 6, 1)], B.default_configs()),   # another block set
                       B.Baoc(blocks, B.default_configs()[:4])):               # another candidate set
        with pytest.raises(B.BaocError) as e:
            bad_handle.import_state(blob)
        assert e.value.code == B.E_INVALID
    for bad_blob in (blob[:10], b"XXXX" + blob[4:]):                           # truncated; foreign magic
        with pytest.raises(B.BaocError) as e:
            B.Baoc(blocks, B.default_configs()).import_state(bad_blob)
        assert e.value.code == B.E_INVALID


def test_options_default_to_the_literal_readings_and_are_validated(B):
    o = B.default_opts()
    assert (o.debias, o.quantizer8, o.use_snr, o.qblock) == (0, B.Q_LINEAR, 1, 256)
    for field, bad in (("debias", 2), ("debias", -1), ("quantizer8", 7), ("qblock", 128)):
        o = B.default_opts()
        setattr(o, field, bad)
        with pytest.raises(B.BaocError) as e:
            B.Baoc([(64, 8, 8)], B.default_configs(), o)
        assert e.value.code == B.E_INVALID
    o = B.default_opts()
    o.debias = 1
    B.Baoc([(64, 8, 8)], B.default_configs(), o)


def test_set_sampling_validates_indices_and_shrinks_the_workspace(B):
    blocks = [(4096 * 8, 256, 128), (1000, 1000, 1)]
    h = B.Baoc(blocks, B.default_configs())
    dense = h.stats_workspace_bytes()
    rows0, cols0 = np.arange(0, 256, 8), np.arange(0, 128, 4)
    h.set_sampling([(rows0, cols0), (np.arange(0, 1000, 10), None)])
    assert h.stats_workspace_bytes() < dense // 3 and h.query().n_tiles == 2     # 64 KB of select histograms per block stay
    assert h.query().stats_bytes_per_call == 26 * (32 * 32 + 100)
    bad = [([0, 0, 3], cols0), ([5, 3], cols0), ([256], cols0), (rows0, [128]), (rows0, None), ([], cols0)]
    for rows, cols in bad:
        with pytest.raises(B.BaocError) as e:
            h.set_sampling([(rows, cols), (np.arange(10), None)])
        assert e.value.code == B.E_INVALID
    with pytest.raises(B.BaocError) as e:
        h.set_sampling([(rows0, cols0), (np.arange(10), np.arange(2))])          # a vector block has one column
    assert e.value.code == B.E_INVALID
    h.set_sampling(None)
    assert h.stats_workspace_bytes() == dense


@pytest.mark.parametrize("seed", range(6))
def test_partition_equals_the_oracle(B, seed):
    """Algorithm 2 in the library against the oracle: the block of every unit and the threshold, bit for bit."""
    rng = np.random.default_rng(100 + seed)
    for trial in range(30):
        m = int(rng.integers(1, 40))
        k = int(rng.integers(1, 6))
        sizes = rng.integers(1, 5000, size=m)
        Z = rng.random((m, k))
        if trial % 3 == 0:                                          # smooth drifts plus jumps: formation merges, the split cuts
            Z = np.cumsum(rng.random((m, k)) * 0.08, axis=0) + (rng.random((m, 1)) < 0.15).cumsum(axis=0) * 0.5
        if trial % 5 == 0:
            Z[rng.integers(0, m)] = Z[0]                            # identical units
        w = None if trial % 2 else rng.random(k) * 2
        alpha = float(rng.choice([0.0, 0.005, 0.03, 0.1, 0.3]))
        tau = None if trial % 4 else float(rng.random() * 0.6)
        want, tau_want = O.partition_blocks(sizes.tolist(), Z, w, alpha, tau)
        got, tau_got = B.partition(sizes, Z, w, alpha, tau)
        assert tau_got == tau_want
        assert got.tolist() == want.tolist(), (seed, trial)


def test_partition_rejects_bad_arguments(B):
    Z = np.zeros((3, 2))
    for bad in (dict(numel=[1, 0, 2]), dict(alpha=-0.1), dict(alpha=1.5), dict(w=[1.0, -1.0]), dict(tau=float("nan"))):
        args = dict(numel=[4, 5, 6], z=Z, w=None, alpha=0.0, tau=None)
        args.update(bad)
        with pytest.raises(B.BaocError):
            B.partition(**args)
    Zbad = Z.copy(); Zbad[1, 1] = np.inf
    with pytest.raises(B.BaocError):
        B.partition([4, 5, 6], Zbad)
    ids, tau = B.partition([7], np.ones((1, 5)))
    assert ids.tolist() == [0] and tau == 0.0
