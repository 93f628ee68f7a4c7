"""Pins for the fp64 CPU oracle: every check here compares it with something that is not
itself -- a hand-worked example, an independently written per-slice loop, closed forms,
invariants and special cases that reduce to numpy / scipy / torch library routines."""
import json
import math
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
from oracle import OracleConfig, ACT_RELU, ACT_GELU_TANH

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rand_weights(rng, cfg, scale=0.5, biases=True):
    ds = cfg.ds
    w = dict(Wr1=rng.normal(0, scale, (cfg.Hr, ds)), Wr2=rng.normal(0, scale, (cfg.E, cfg.Hr)),
             W1=rng.normal(0, scale, (cfg.E, cfg.F, ds)), W2=rng.normal(0, scale, (cfg.E, ds, cfg.F)))
    if biases:
        w.update(br1=rng.normal(0, scale, cfg.Hr), br2=rng.normal(0, scale, cfg.E),
                 b1=rng.normal(0, scale, (cfg.E, cfg.F)), b2=rng.normal(0, scale, (cfg.E, ds)))
    return w


def identity_expert(ds, F):
    """ReLU FFN with W1 = [I; -I; 0], W2 = [I, -I, 0]: relu(z) - relu(-z) = z."""
    assert F >= 2 * ds
    W1 = np.zeros((F, ds))
    W2 = np.zeros((ds, F))
    W1[:ds] = np.eye(ds)
    W1[ds:2 * ds] = -np.eye(ds)
    W2[:, :ds] = np.eye(ds)
    W2[:, ds:2 * ds] = -np.eye(ds)
    return W1, W2


# ---------------------------------------------------------------------------------------------
# Section 3.1 + Eq. 1: hand-worked example with exact rational results
# ---------------------------------------------------------------------------------------------
def test_handworked_example():
    g = json.load(open(os.path.join(GOLDEN, "handworked_layer.json")))
    cfg = OracleConfig(T=g["T"], d=g["d"], S=g["S"], E=g["E"], k=g["k"], Hr=g["Hr"], F=g["F"],
                       act=ACT_RELU)
    w = dict(Wr1=np.array(g["Wr1"]), Wr2=np.log(np.array(g["Wr2_log_of"])),
             W1=np.array(g["W1"]), b1=np.array(g["b1"]), W2=np.array(g["W2"]), b2=np.array(g["b2"]))
    out = oracle.forward(cfg, np.array(g["h"]), w)
    probs = np.array([[n / d for n, d in row] for row in g["expect_probs_fractions"]])
    h_out = np.array([n / d for n, d in g["expect_h_out_fractions"]])
    np.testing.assert_allclose(out["probs"], probs, rtol=0, atol=1e-15)
    assert out["topk_idx"].tolist() == g["expect_topk_idx"]
    assert out["assigned"].tolist() == g["expect_assigned"]
    np.testing.assert_allclose(out["h_out"].ravel(), h_out, rtol=0, atol=1e-14)
    # the gate sits on the expert's input: gating the output instead would give another number
    wrong = 16 / 19 * (2 * 1 + 2 + 1 + 2 * 2 - 1 + 0.5) + 3 / 19 * 1
    assert abs(out["h_out"][0, 0] - wrong) > 0.05


# ---------------------------------------------------------------------------------------------
# Brute force: an independent per-slice loop in plain Python (no grouping, no offsets)
# ---------------------------------------------------------------------------------------------
def brute_force_layer(cfg, h, w):
    ds = cfg.ds
    T, S, E, k = cfg.T, cfg.S, cfg.E, cfg.k
    out = [[0.0] * cfg.d for _ in range(T)]
    chosen = {}
    probs_all = {}
    for t in range(T):
        for s in range(S):
            x = [float(h[t][s * ds + q]) for q in range(ds)]
            hidden = []
            for i in range(cfg.Hr):
                z = math.fsum(float(w["Wr1"][i][q]) * x[q] for q in range(ds))
                z += float(w["br1"][i]) if "br1" in w else 0.0
                hidden.append(max(z, 0.0))
            logits = []
            for e in range(E):
                z = math.fsum(float(w["Wr2"][e][i]) * hidden[i] for i in range(cfg.Hr))
                z += float(w["br2"][e]) if "br2" in w else 0.0
                logits.append(z)
            top = max(logits)
            ex = [math.exp(z - top) for z in logits]
            den = math.fsum(ex)
            p = [v / den for v in ex]
            order = sorted(range(E), key=lambda e: (-p[e], e))[:k]
            chosen[(t, s)] = order
            probs_all[(t, s)] = p
    # capacity: walk pairs in (token, slice, j) order
    taken = [0] * E
    keep = {}
    for t in range(T):
        for s in range(S):
            for j, e in enumerate(chosen[(t, s)]):
                keep[(t, s, j)] = (cfg.capacity == 0) or (taken[e] < cfg.capacity)
                taken[e] += 1
    for t in range(T):
        for s in range(S):
            x = [float(h[t][s * ds + q]) for q in range(ds)]
            p = probs_all[(t, s)]
            for j, e in enumerate(chosen[(t, s)]):
                if not keep[(t, s, j)]:
                    continue
                xt = [p[e] * v for v in x]
                u = []
                for f in range(cfg.F):
                    z = math.fsum(float(w["W1"][e][f][q]) * xt[q] for q in range(ds))
                    z += float(w["b1"][e][f]) if "b1" in w else 0.0
                    if cfg.act == ACT_RELU:
                        u.append(max(z, 0.0))
                    else:
                        u.append(0.5 * z * (1.0 + math.tanh(math.sqrt(2.0 / math.pi) * (z + 0.044715 * z ** 3))))
                for q in range(ds):
                    y = math.fsum(float(w["W2"][e][q][f]) * u[f] for f in range(cfg.F))
                    y += float(w["b2"][e][q]) if "b2" in w else 0.0
                    out[t][s * ds + q] += y
    return np.array(out), chosen, taken


@pytest.mark.parametrize("shape", [
    dict(T=3, d=8, S=2, E=3, k=2, Hr=5, F=4, act=ACT_RELU, capacity=0),
    dict(T=4, d=12, S=3, E=4, k=3, Hr=7, F=6, act=ACT_GELU_TANH, capacity=0),
    dict(T=5, d=6, S=2, E=3, k=1, Hr=4, F=5, act=ACT_GELU_TANH, capacity=2),
    dict(T=6, d=4, S=1, E=2, k=2, Hr=3, F=3, act=ACT_RELU, capacity=5),
])
@pytest.mark.parametrize("seed", [0, 1])
def test_matches_brute_force(shape, seed):
    cfg = OracleConfig(**shape)
    rng = np.random.default_rng(seed)
    h = rng.normal(0, 1, (cfg.T, cfg.d))
    w = rand_weights(rng, cfg, biases=(seed == 0))
    out = oracle.forward(cfg, h, w)
    ref, chosen, taken = brute_force_layer(cfg, h, w)
    np.testing.assert_allclose(out["h_out"], ref, rtol=1e-12, atol=1e-13)
    for t in range(cfg.T):
        for s in range(cfg.S):
            assert out["topk_idx"][t * cfg.S + s].tolist() == chosen[(t, s)]
    assert out["assigned"].tolist() == taken


# ---------------------------------------------------------------------------------------------
# Invariants of routing and grouping
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("capacity", [0, 40])
def test_invariants(capacity):
    cfg = OracleConfig(T=37, d=24, S=3, E=7, k=3, Hr=16, F=10, act=ACT_GELU_TANH, capacity=capacity)
    rng = np.random.default_rng(5)
    h = rng.normal(0, 1, (cfg.T, cfg.d))
    w = rand_weights(rng, cfg)
    out = oracle.forward(cfg, h, w)
    np.testing.assert_allclose(out["probs"].sum(axis=1), 1.0, rtol=0, atol=1e-14)
    idx = out["topk_idx"]
    assert all(len(set(r)) == cfg.k for r in idx.tolist())               # k distinct experts per slice
    assert out["assigned"].sum() == cfg.T * cfg.S * cfg.k                  # Section 3.2: B*S*k decisions
    assert np.all(np.diff(out["topk_p"], axis=1) <= 0)                     # most probable first
    assert np.all(out["gap"] >= 0)
    dest = out["dest"]
    kept = out["kept"]
    assert kept.sum() == (dest >= 0).sum()
    if capacity:
        assert np.all(kept <= capacity)
        assert np.all(kept == np.minimum(out["assigned"], capacity))
    else:
        assert np.all(kept == out["assigned"])
    live = np.sort(dest[dest >= 0])
    assert np.array_equal(live, np.arange(kept.sum()))                    # bijection onto [0, sum kept)
    np.testing.assert_array_equal(out["offsets"], np.concatenate([[0], np.cumsum(kept)]))
    flat_idx, flat_dest = idx.ravel(), dest.ravel()
    for e in range(cfg.E):
        d_e = flat_dest[flat_idx == e]
        d_live = d_e[d_e >= 0]
        assert np.all(np.diff(d_live) == 1)                                # stable: increasing in (n, j)
        assert np.all(d_e[:len(d_live)] >= 0) and np.all(d_e[len(d_live):] < 0)  # first come, first kept
        if len(d_live):
            assert d_live[0] == out["offsets"][e]


# ---------------------------------------------------------------------------------------------
# Identity experts (ReLU): h' = p_top * h slice-wise for k = 1; h' = h for E = 1
# ---------------------------------------------------------------------------------------------
def test_identity_experts_k1_gives_p_times_h():
    cfg = OracleConfig(T=9, d=12, S=3, E=4, k=1, Hr=8, F=8, act=ACT_RELU)
    rng = np.random.default_rng(2)
    h = rng.normal(0, 1, (cfg.T, cfg.d))
    w = rand_weights(rng, cfg, biases=False)
    W1, W2 = identity_expert(cfg.ds, cfg.F)
    w["W1"] = np.stack([W1] * cfg.E)
    w["W2"] = np.stack([W2] * cfg.E)
    out = oracle.forward(cfg, h, w)
    p_top = out["probs"].max(axis=1)
    expect = (h.reshape(cfg.N, cfg.ds) * p_top[:, None]).reshape(cfg.T, cfg.d)
    np.testing.assert_allclose(out["h_out"], expect, rtol=1e-14, atol=1e-15)
    np.testing.assert_array_equal(out["topk_idx"][:, 0], out["probs"].argmax(axis=1))


def test_single_identity_expert_returns_h():
    cfg = OracleConfig(T=5, d=8, S=2, E=1, k=1, Hr=4, F=8, act=ACT_RELU)
    rng = np.random.default_rng(3)
    h = rng.normal(0, 1, (cfg.T, cfg.d))
    w = rand_weights(rng, cfg, biases=False)
    W1, W2 = identity_expert(cfg.ds, cfg.F)
    w["W1"], w["W2"] = W1[None], W2[None]
    out = oracle.forward(cfg, h, w)
    np.testing.assert_array_equal(out["probs"], np.ones((cfg.N, 1)))
    np.testing.assert_allclose(out["h_out"], h, rtol=0, atol=1e-15)
    assert np.all(np.isinf(out["gap"]))


# ---------------------------------------------------------------------------------------------
# S = 1 is token-level MoE, and slicing is a free reshape
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("capacity", [0, 11])
def test_slices_are_rows_of_a_reshape(capacity):
    cfg = OracleConfig(T=10, d=24, S=4, E=5, k=2, Hr=9, F=7, act=ACT_GELU_TANH, capacity=capacity)
    flat = OracleConfig(T=cfg.T * cfg.S, d=cfg.ds, S=1, E=5, k=2, Hr=9, F=7, act=ACT_GELU_TANH,
                        capacity=capacity)
    rng = np.random.default_rng(4)
    h = rng.normal(0, 1, (cfg.T, cfg.d))
    w = rand_weights(rng, cfg)
    a = oracle.forward(cfg, h, w)
    b = oracle.forward(flat, h.reshape(flat.T, flat.d), w)
    np.testing.assert_array_equal(a["h_out"].reshape(flat.T, flat.d), b["h_out"])
    np.testing.assert_array_equal(a["topk_idx"], b["topk_idx"])
    np.testing.assert_array_equal(a["dest"], b["dest"])


def test_token_level_moe_against_numpy_and_scipy():
    """S = 1: logits, softmax and the gated experts re-done with numpy matmul / scipy softmax."""
    from scipy.special import softmax
    cfg = OracleConfig(T=16, d=6, S=1, E=4, k=2, Hr=5, F=9, act=ACT_RELU)
    rng = np.random.default_rng(8)
    h = rng.normal(0, 1, (cfg.T, cfg.d))
    w = rand_weights(rng, cfg)
    out = oracle.forward(cfg, h, w)
    logits = np.maximum(h @ w["Wr1"].T + w["br1"], 0) @ w["Wr2"].T + w["br2"]
    p = softmax(logits, axis=1)
    np.testing.assert_allclose(out["probs"], p, rtol=1e-13, atol=1e-15)
    order = np.argsort(-p, axis=1, kind="stable")[:, :cfg.k]
    np.testing.assert_array_equal(out["topk_idx"], order)
    expect = np.zeros_like(h)
    for t in range(cfg.T):
        for e in order[t]:
            u = np.maximum(w["W1"][e] @ (p[t, e] * h[t]) + w["b1"][e], 0)
            expect[t] += w["W2"][e] @ u + w["b2"][e]
    np.testing.assert_allclose(out["h_out"], expect, rtol=1e-12, atol=1e-13)


# ---------------------------------------------------------------------------------------------
# Zero router: p = 1/E, ties go to the lowest ids; capacity keeps the first C rows
# ---------------------------------------------------------------------------------------------
def test_zero_router_ties_and_capacity():
    cfg = OracleConfig(T=12, d=8, S=2, E=5, k=2, Hr=4, F=8, act=ACT_RELU, capacity=7)
    rng = np.random.default_rng(6)
    h = rng.normal(0, 1, (cfg.T, cfg.d))
    w = rand_weights(rng, cfg, biases=False)
    w["Wr1"] = np.zeros_like(w["Wr1"])
    w["Wr2"] = np.zeros_like(w["Wr2"])
    W1, W2 = identity_expert(cfg.ds, cfg.F)
    w["W1"], w["W2"] = np.stack([W1] * cfg.E), np.stack([W2] * cfg.E)
    out = oracle.forward(cfg, h, w)
    np.testing.assert_allclose(out["probs"], 1.0 / cfg.E, rtol=0, atol=1e-16)
    assert np.all(out["topk_idx"] == np.array([0, 1]))
    assert out["assigned"].tolist() == [cfg.N, cfg.N, 0, 0, 0]
    assert out["kept"].tolist() == [7, 7, 0, 0, 0]
    # rows n < 7 keep both experts (identity, gate 1/5 each): h' = 2/5 h; the rest become zero
    x = h.reshape(cfg.N, cfg.ds)
    expect = np.zeros_like(x)
    expect[:7] = 2.0 / cfg.E * x[:7]
    np.testing.assert_allclose(out["h_out"].reshape(cfg.N, cfg.ds), expect, rtol=1e-14, atol=1e-16)
    assert np.all(out["gap"] == 0.0)


def test_zipf_bias_sends_everything_to_expert_zero():
    """Router output bias 1.5*log(Zipf weight), k = 1, zero router weights: softmax of the bias
    alone (p_e proportional to w_e^1.5), every slice on expert 0, first C rows kept."""
    E, s = 6, 1.2
    cfg = OracleConfig(T=10, d=6, S=2, E=E, k=1, Hr=3, F=6, act=ACT_RELU, capacity=8)
    rng = np.random.default_rng(7)
    h = rng.normal(0, 1, (cfg.T, cfg.d))
    w = rand_weights(rng, cfg, biases=False)
    w["Wr1"] = np.zeros_like(w["Wr1"])
    zw = np.arange(1, E + 1.0) ** (-s)
    zw /= zw.sum()
    w["br2"] = 1.5 * np.log(zw)
    W1, W2 = identity_expert(cfg.ds, cfg.F)
    w["W1"], w["W2"] = np.stack([W1] * E), np.stack([W2] * E)
    out = oracle.forward(cfg, h, w)
    p_expect = zw ** 1.5 / (zw ** 1.5).sum()
    np.testing.assert_allclose(out["probs"], np.tile(p_expect, (cfg.N, 1)), rtol=1e-13)
    assert np.all(out["topk_idx"] == 0)
    assert out["assigned"].tolist() == [cfg.N] + [0] * (E - 1)
    assert out["kept"].tolist() == [8] + [0] * (E - 1)
    x = h.reshape(cfg.N, cfg.ds)
    expect = np.zeros_like(x)
    expect[:8] = p_expect[0] * x[:8]
    np.testing.assert_allclose(out["h_out"].reshape(cfg.N, cfg.ds), expect, rtol=1e-13, atol=1e-16)
    np.testing.assert_array_equal(out["dest"].ravel(), np.r_[np.arange(8), -np.ones(cfg.N - 8)])


# ---------------------------------------------------------------------------------------------
# Equivariance: shared router and position-free experts (Section 3.1)
# ---------------------------------------------------------------------------------------------
def test_token_and_slice_permutation_equivariance():
    cfg = OracleConfig(T=8, d=12, S=3, E=4, k=2, Hr=6, F=5, act=ACT_GELU_TANH)
    rng = np.random.default_rng(9)
    h = rng.normal(0, 1, (cfg.T, cfg.d))
    w = rand_weights(rng, cfg)
    base = oracle.forward(cfg, h, w)["h_out"]
    tp = rng.permutation(cfg.T)
    np.testing.assert_array_equal(oracle.forward(cfg, h[tp], w)["h_out"], base[tp])
    sp = rng.permutation(cfg.S)
    hs = h.reshape(cfg.T, cfg.S, cfg.ds)[:, sp].reshape(cfg.T, cfg.d)
    expect = base.reshape(cfg.T, cfg.S, cfg.ds)[:, sp].reshape(cfg.T, cfg.d)
    np.testing.assert_array_equal(oracle.forward(cfg, hs, w)["h_out"], expect)


# ---------------------------------------------------------------------------------------------
# Affine special case: large positive b1 keeps every ReLU open
# ---------------------------------------------------------------------------------------------
def test_affine_special_case_with_one_matvec():
    cfg = OracleConfig(T=6, d=10, S=2, E=3, k=2, Hr=4, F=7, act=ACT_RELU)
    rng = np.random.default_rng(10)
    h = rng.normal(0, 1, (cfg.T, cfg.d))
    w = rand_weights(rng, cfg)
    w["b1"] = np.full((cfg.E, cfg.F), 100.0)
    out = oracle.forward(cfg, h, w)
    x = h.reshape(cfg.N, cfg.ds)
    expect = np.zeros_like(x)
    for n in range(cfg.N):
        for e in out["topk_idx"][n]:
            p = out["probs"][n, e]
            expect[n] += p * (w["W2"][e] @ w["W1"][e]) @ x[n] + w["W2"][e] @ w["b1"][e] + w["b2"][e]
    np.testing.assert_allclose(out["h_out"].reshape(cfg.N, cfg.ds), expect, rtol=1e-11, atol=1e-11)


# ---------------------------------------------------------------------------------------------
# E = 1, k = 1: a plain two-layer MLP; GELU(tanh) against torch's library routine
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("act", [ACT_RELU, ACT_GELU_TANH])
def test_single_expert_is_a_dense_mlp(act):
    torch = pytest.importorskip("torch")
    cfg = OracleConfig(T=20, d=16, S=2, E=1, k=1, Hr=4, F=12, act=act)
    rng = np.random.default_rng(11)
    h = rng.normal(0, 1, (cfg.T, cfg.d))
    w = rand_weights(rng, cfg)
    out = oracle.forward(cfg, h, w)
    x = torch.from_numpy(h.reshape(cfg.N, cfg.ds))
    z = x @ torch.from_numpy(w["W1"][0]).T + torch.from_numpy(w["b1"][0])
    u = torch.relu(z) if act == ACT_RELU else torch.nn.functional.gelu(z, approximate="tanh")
    y = u @ torch.from_numpy(w["W2"][0]).T + torch.from_numpy(w["b2"][0])
    np.testing.assert_allclose(out["h_out"].reshape(cfg.N, cfg.ds), y.numpy(), rtol=1e-12, atol=1e-13)


# ---------------------------------------------------------------------------------------------
# Staged calls, forced routing and sampled rows agree with the whole-layer call
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("capacity", [0, 9])
def test_staged_calls_compose_to_forward(capacity):
    cfg = OracleConfig(T=11, d=12, S=3, E=6, k=2, Hr=8, F=9, act=ACT_GELU_TANH, capacity=capacity)
    rng = np.random.default_rng(12)
    h = rng.normal(0, 1, (cfg.T, cfg.d))
    w = rand_weights(rng, cfg)
    full = oracle.forward(cfg, h, w)
    r = oracle.route(cfg, h, w)
    np.testing.assert_array_equal(r["topk_idx"], full["topk_idx"])
    np.testing.assert_array_equal(r["probs"], full["probs"])
    d = oracle.dispatch(cfg, r["topk_idx"])
    np.testing.assert_array_equal(d["dest"], full["dest"])
    np.testing.assert_array_equal(d["kept"], full["kept"])
    # perm inverts dest on the kept pairs
    flat_dest = d["dest"].ravel()
    np.testing.assert_array_equal(flat_dest[d["perm"]], np.arange(d["kept"].sum()))
    n_kept = int(d["offsets"][-1])
    xperm = oracle.weight_slices(cfg, h, r["topk_p"], d["dest"], n_kept)
    # Eq. 1, row by row through perm
    x = h.reshape(cfg.N, cfg.ds)
    for row, pair in enumerate(d["perm"]):
        np.testing.assert_array_equal(xperm[row], r["topk_p"].ravel()[pair] * x[pair // cfg.k])
    yperm = oracle.expert_ffn(cfg, xperm, d["offsets"], w)
    h_out = oracle.combine(cfg, yperm, d["dest"])
    np.testing.assert_array_equal(h_out, full["h_out"])


def test_forced_routing():
    cfg = OracleConfig(T=9, d=8, S=2, E=5, k=2, Hr=6, F=7, act=ACT_GELU_TANH)
    rng = np.random.default_rng(13)
    h = rng.normal(0, 1, (cfg.T, cfg.d))
    w = rand_weights(rng, cfg)
    free = oracle.forward(cfg, h, w)
    same = oracle.forward(cfg, h, w, forced_idx=free["topk_idx"])
    np.testing.assert_array_equal(same["h_out"], free["h_out"])
    swapped = oracle.forward(cfg, h, w, forced_idx=free["topk_idx"][:, ::-1])
    np.testing.assert_allclose(swapped["h_out"], free["h_out"], rtol=1e-14, atol=1e-15)
    np.testing.assert_array_equal(swapped["topk_p"], free["topk_p"][:, ::-1])
    # forcing other experts changes the gates to those experts' probabilities
    other = (free["topk_idx"] + 1) % cfg.E
    forced = oracle.forward(cfg, h, w, forced_idx=other)
    np.testing.assert_array_equal(forced["topk_p"], np.take_along_axis(free["probs"], other, axis=1))
    assert np.array_equal(forced["assigned"], np.bincount(other.ravel(), minlength=cfg.E))


@pytest.mark.parametrize("capacity", [0, 10])
def test_sampled_rows_match_forward(capacity):
    cfg = OracleConfig(T=13, d=12, S=3, E=4, k=2, Hr=6, F=7, act=ACT_GELU_TANH, capacity=capacity)
    rng = np.random.default_rng(14)
    h = rng.normal(0, 1, (cfg.T, cfg.d))
    w = rand_weights(rng, cfg)
    full = oracle.forward(cfg, h, w)
    pick = rng.choice(cfg.N, 17, replace=False)
    got = oracle.rows(cfg, h, w, pick, full["topk_idx"][pick], (full["dest"][pick] >= 0))
    np.testing.assert_allclose(got["y"], full["h_out"].reshape(cfg.N, cfg.ds)[pick], rtol=1e-15, atol=1e-16)
    np.testing.assert_array_equal(got["p"], full["topk_p"][pick])


# ---------------------------------------------------------------------------------------------
# Eq. 2 and ELE closed forms
# ---------------------------------------------------------------------------------------------
def test_load_stats_closed_forms():
    l_cap, ele = oracle.load_stats([5, 5, 5, 5], alpha=0.1)
    assert l_cap == 0.0 and abs(ele - 1.0) < 1e-15
    l_cap, ele = oracle.load_stats([12, 0, 0, 0], alpha=0.1)
    assert ele == 0.0
    assert abs(l_cap - 0.1 * 3.0) < 1e-15          # CV^2 of a one-hot over E is E - 1
    counts = np.array([1, 2, 3, 10])
    l_cap, ele = oracle.load_stats(counts, alpha=0.05)
    assert abs(l_cap - 0.05 * (np.std(counts) / np.mean(counts)) ** 2) < 1e-15
    from scipy.stats import entropy
    assert abs(ele - entropy(counts / counts.sum()) / math.log(4)) < 1e-14
    # exact values: loads 1/2, 1/4, 1/4 -> entropy 1.5 bits
    l_cap, ele = oracle.load_stats([2, 1, 1], alpha=1.0)
    assert abs(ele - 1.5 / math.log2(3)) < 1e-15
    assert abs(l_cap - float(Fraction(2, 9) / Fraction(16, 9))) < 1e-15
