"""Pins for the oracle's backward pass (Section 3.1: router and experts are trained end to end).

The paper prints no gradient formulas, so the backward is pinned to things that do not share its
hand-written chain rule: central finite differences of the separately pinned forward, torch's
reverse-mode differentiation of an independently written fp64 forward, and closed forms."""
import numpy as np
import pytest
import torch

import oracle
from oracle import OracleConfig, ACT_RELU, ACT_GELU_TANH

GRADS = ("dh", "dWr1", "dbr1", "dWr2", "dbr2", "dW1", "db1", "dW2", "db2")
PARAM_OF = dict(dWr1="Wr1", dbr1="br1", dWr2="Wr2", dbr2="br2", dW1="W1", db1="b1", dW2="W2", db2="b2")


def make_case(seed, T=6, d=12, S=3, E=4, k=2, Hr=8, F=10, act=ACT_GELU_TANH, capacity=0,
              temperature=0.0, biases=True, scale=0.6):
    rng = np.random.default_rng(seed)
    cfg = OracleConfig(T=T, d=d, S=S, E=E, k=k, Hr=Hr, F=F, act=act, capacity=capacity,
                       temperature=temperature)
    ds = cfg.ds
    w = dict(Wr1=rng.normal(0, scale, (Hr, ds)), Wr2=rng.normal(0, scale, (E, Hr)),
             W1=rng.normal(0, scale, (E, F, ds)), W2=rng.normal(0, scale, (E, ds, F)))
    if biases:
        w.update(br1=rng.normal(0, scale, Hr), br2=rng.normal(0, scale, E),
                 b1=rng.normal(0, scale, (E, F)), b2=rng.normal(0, scale, (E, ds)))
    h = rng.normal(0, 1, (T, d))
    gout = rng.normal(0, 1, (T, d))
    return cfg, h, w, gout


# ---------------------------------------------------------------------------------------------
# reverse-mode differentiation by torch of a forward written here in plain tensor ops
# ---------------------------------------------------------------------------------------------
def torch_grads(cfg, h, w, gout, idx, dest, dropped=None):
    """L = <gout, h'> with h' from Section 3.1 / Eq. 1 on fixed expert ids; grads by autograd."""
    t = {n: torch.tensor(np.asarray(v), dtype=torch.float64, requires_grad=True) for n, v in w.items()}
    x = torch.tensor(h, dtype=torch.float64, requires_grad=True)
    X = x.reshape(cfg.N, cfg.ds)
    tau = cfg.temperature if cfg.temperature > 0 else 1.0
    pre = X @ t["Wr1"].T + (t["br1"] if "br1" in t else 0.0)
    logits = torch.relu(pre) @ t["Wr2"].T + (t["br2"] if "br2" in t else 0.0)
    p = torch.softmax(logits / tau, dim=1)
    rows = []
    for n in range(cfg.N):
        y = torch.zeros(cfg.ds, dtype=torch.float64)
        gates = [p[n, int(idx[n, j])] for j in range(cfg.k)]
        if dropped is not None:     # Section 3.3: survivors re-normalised; all dropped -> top-1 gets 1
            alive = [j for j in range(cfg.k) if not dropped[n, j]]
            total = sum(gates[j] for j in alive) if alive else None
            gates = [(gates[j] / total if j in alive else torch.tensor(0.0, dtype=torch.float64)) if alive
                     else torch.tensor(1.0 if j == 0 else 0.0, dtype=torch.float64) for j in range(cfg.k)]
        for j in range(cfg.k):
            if dest[n, j] < 0:
                continue
            e = int(idx[n, j])
            z = t["W1"][e] @ (gates[j] * X[n]) + (t["b1"][e] if "b1" in t else 0.0)
            u = torch.relu(z) if cfg.act == ACT_RELU else torch.nn.functional.gelu(z, approximate="tanh")
            y = y + t["W2"][e] @ u + (t["b2"][e] if "b2" in t else 0.0)
        rows.append(y)
    hp = torch.stack(rows).reshape(cfg.T, cfg.d)
    loss = (hp * torch.tensor(gout, dtype=torch.float64)).sum()
    loss.backward()
    out = dict(dh=x.grad.numpy())
    for g, name in PARAM_OF.items():
        if name in t:
            out[g] = np.zeros(t[name].shape) if t[name].grad is None else t[name].grad.numpy()
    return out, hp.detach().numpy()


@pytest.mark.parametrize("kw", [
    dict(seed=1),
    dict(seed=2, act=ACT_RELU),
    dict(seed=3, k=1, E=3),
    dict(seed=4, k=3, E=5),
    dict(seed=5, capacity=5),                  # some pairs are dropped
    dict(seed=6, temperature=2.5),
    dict(seed=7, biases=False, temperature=0.5),
    dict(seed=8, S=1, d=8, T=9),               # token-level MoE
])
def test_backward_matches_autograd(kw):
    cfg, h, w, gout = make_case(**kw)
    fwd = oracle.forward(cfg, h, w)
    ref, hp = torch_grads(cfg, h, w, gout, fwd["topk_idx"], fwd["dest"])
    np.testing.assert_allclose(hp, fwd["h_out"], rtol=0, atol=1e-12)   # same function
    got = oracle.backward(cfg, h, w, gout)
    if cfg.capacity:
        assert (fwd["dest"] < 0).any() and (fwd["dest"] >= 0).any()
    for g in GRADS:
        if g in ref:
            scale = max(1.0, np.abs(ref[g]).max())
            np.testing.assert_allclose(got[g], ref[g], rtol=0, atol=1e-11 * scale, err_msg=g)


# ---------------------------------------------------------------------------------------------
# central finite differences of the oracle's own (pinned) forward, routing held fixed
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("kw", [dict(seed=11), dict(seed=12, act=ACT_RELU, capacity=6),
                                dict(seed=13, k=1, temperature=1.7)])
def test_backward_matches_finite_differences(kw):
    cfg, h, w, gout = make_case(**kw)
    idx = oracle.forward(cfg, h, w)["topk_idx"]
    got = oracle.backward(cfg, h, w, gout, forced_idx=idx)
    rng = np.random.default_rng(99)

    def loss(hh, ww):
        return float((oracle.forward(cfg, hh, ww, forced_idx=idx)["h_out"] * gout).sum())

    eps = 1e-5
    for g in GRADS:
        name = "h" if g == "dh" else PARAM_OF[g]
        base = h if g == "dh" else w[name]
        for _ in range(6):
            pos = tuple(int(rng.integers(0, s)) for s in base.shape)
            hi, lo = base.copy(), base.copy()
            hi[pos] += eps
            lo[pos] -= eps
            if g == "dh":
                fd = (loss(hi, w) - loss(lo, w)) / (2 * eps)
            else:
                fd = (loss(h, {**w, name: hi}) - loss(h, {**w, name: lo})) / (2 * eps)
            # ReLU kinks can sit inside the stencil; 1e-5 steps make that vanishingly rare here
            assert abs(fd - got[g][pos]) <= 2e-6 * max(1.0, abs(fd)), (g, pos, fd, got[g][pos])


# ---------------------------------------------------------------------------------------------
# closed forms and invariants
# ---------------------------------------------------------------------------------------------
def test_single_expert_router_gets_no_gradient():
    """E = 1: p = 1 whatever the router does, so the router's gradients vanish and dh is the
    expert's own input gradient."""
    cfg, h, w, gout = make_case(21, E=1, k=1)
    got = oracle.backward(cfg, h, w, gout)
    for g in ("dWr1", "dbr1", "dWr2", "dbr2"):
        assert np.abs(got[g]).max() == 0.0
    X, G = h.reshape(cfg.N, cfg.ds), gout.reshape(cfg.N, cfg.ds)
    z = X @ w["W1"][0].T + w["b1"][0]
    zt = torch.tensor(z, requires_grad=True)
    torch.nn.functional.gelu(zt, approximate="tanh").sum().backward()
    dx = ((G @ w["W2"][0]) * zt.grad.numpy()) @ w["W1"][0]
    np.testing.assert_allclose(got["dh"].reshape(cfg.N, cfg.ds), dx, atol=1e-12)
    np.testing.assert_allclose(got["db2"][0], G.sum(0), atol=1e-12)


def test_shifted_identity_expert():
    """E = 1, ReLU expert with W1 = W2 = I and a first bias large enough to keep every unit
    active: h' = h + b1 + b2, hence dh = gout, db1 = db2 = column sums of gout."""
    T, d, S = 5, 8, 2
    ds = d // S
    cfg = OracleConfig(T=T, d=d, S=S, E=1, k=1, Hr=3, F=ds, act=ACT_RELU)
    rng = np.random.default_rng(5)
    h, gout = rng.normal(0, 1, (T, d)), rng.normal(0, 1, (T, d))
    w = dict(Wr1=rng.normal(0, 1, (3, ds)), Wr2=rng.normal(0, 1, (1, 3)),
             W1=np.eye(ds)[None], b1=np.full((1, ds), 100.0), W2=np.eye(ds)[None], b2=np.ones((1, ds)))
    got = oracle.backward(cfg, h, w, gout)
    G = gout.reshape(-1, ds)
    np.testing.assert_allclose(got["dh"], gout, atol=1e-13)
    np.testing.assert_allclose(got["db1"][0], G.sum(0), atol=1e-12)
    np.testing.assert_allclose(got["db2"][0], G.sum(0), atol=1e-12)
    np.testing.assert_allclose(got["dW2"][0], G.T @ (h.reshape(-1, ds) + 100.0), atol=1e-10)
    np.testing.assert_allclose(got["dW1"][0], G.T @ h.reshape(-1, ds), atol=1e-12)


def test_softmax_jacobian_invariants():
    """The softmax does not change when a constant is added to all logits: the logit gradients of
    a row sum to zero, so dbr2 sums to zero and the columns of dWr2 sum to zero."""
    cfg, h, w, gout = make_case(31, E=6, k=2)
    got = oracle.backward(cfg, h, w, gout)
    assert np.abs(got["dbr2"]).max() > 1e-3
    assert abs(got["dbr2"].sum()) < 1e-12
    assert np.abs(got["dWr2"].sum(axis=0)).max() < 1e-12


def test_dropped_slices_receive_no_gradient():
    """Zero router weights send every slice to expert 0 (ties go to the lowest id); a capacity of
    C keeps the first C slices.  The others add nothing to h', so their dh is zero, and experts
    that saw no slice have zero gradients."""
    cfg, h, w, gout = make_case(41, T=8, S=2, d=8, E=3, k=1, capacity=5)
    w["Wr1"][:] = 0
    w["Wr2"][:] = 0
    w["br1"][:] = 0
    w["br2"][:] = 0
    got = oracle.backward(cfg, h, w, gout)
    dX = got["dh"].reshape(cfg.N, cfg.ds)
    assert np.abs(dX[:5]).min() > 0 and np.abs(dX[5:]).max() == 0.0
    assert np.abs(got["dW1"][1:]).max() == 0.0 and np.abs(got["db2"][1:]).max() == 0.0
    np.testing.assert_allclose(got["db2"][0], gout.reshape(cfg.N, cfg.ds)[:5].sum(0), atol=1e-13)


def test_gate_path_by_hand_for_one_row():
    """k = 1, one row: the gate is the only way to the router, so the logit gradients are
    p_e (1 - p_e) <W1^T dz, x> for the chosen expert e and -p_m p_e <W1^T dz, x> for the others,
    worked out here by hand."""
    cfg, h, w, gout = make_case(51, T=1, S=1, d=4, E=3, k=1, Hr=5, F=6, act=ACT_RELU)
    fwd = oracle.forward(cfg, h, w)
    e, p = int(fwd["topk_idx"][0, 0]), fwd["probs"][0]
    x, dy = h[0], gout[0]
    z = w["W1"][e] @ (p[e] * x) + w["b1"][e]
    dz = (w["W2"][e].T @ dy) * (z > 0)
    dpe = float((w["W1"][e].T @ dz) @ x)
    dg = -p * p[e] * dpe
    dg[e] = p[e] * (1 - p[e]) * dpe
    got = oracle.backward(cfg, h, w, gout)
    np.testing.assert_allclose(got["dbr2"], dg, atol=1e-13)


def test_forced_routing_matches_own_routing():
    cfg, h, w, gout = make_case(61)
    idx = oracle.forward(cfg, h, w)["topk_idx"]
    a, b = oracle.backward(cfg, h, w, gout), oracle.backward(cfg, h, w, gout, forced_idx=idx)
    for g in GRADS:
        assert np.array_equal(a[g], b[g])


# ---------------------------------------------------------------------------------------------
# train mode: the gates of cross-slice dropout (Section 3.3) inside the backward
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("kw,rate", [(dict(seed=71, T=10), 0.4), (dict(seed=72, k=3, E=6, T=10), 0.5),
                                      (dict(seed=73, capacity=6, T=10), 0.3), (dict(seed=74), 0.0),
                                      (dict(seed=75, k=1, E=3, T=12), 0.5)])
def test_dropout_gates_backward_matches_autograd(kw, rate):
    cfg, h, w, gout = make_case(**kw)
    fwd = oracle.forward(cfg, h, w)
    gates, dropped = oracle.gate_dropout(fwd["topk_p"], seed=5, rate=rate)
    if rate > 0:
        assert dropped.any() and (~dropped).any()
        if cfg.k > 1:
            assert dropped.all(axis=1).any() or rate < 0.5   # the all-dropped rule is usually exercised
    ref, hp = torch_grads(cfg, h, w, gout, fwd["topk_idx"], fwd["dest"], dropped)
    # the function differentiated is the staged train-mode chain of the oracle
    xperm = oracle.weight_slices(cfg, h, gates, fwd["dest"], int(fwd["offsets"][-1]))
    chain = oracle.combine(cfg, oracle.expert_ffn(cfg, xperm, fwd["offsets"], w), fwd["dest"])
    np.testing.assert_allclose(hp, chain, rtol=0, atol=1e-12)
    got = oracle.backward(cfg, h, w, gout, dropped=dropped)
    for g in GRADS:
        if g in ref:
            scale = max(1.0, np.abs(ref[g]).max())
            np.testing.assert_allclose(got[g], ref[g], rtol=0, atol=1e-11 * scale, err_msg=g)


def test_dropout_rate_zero_differs_from_plain_gates():
    """Rate 0 still re-normalises the k probabilities, so its gradients are not the inference ones."""
    cfg, h, w, gout = make_case(81)
    none = np.zeros((cfg.N, cfg.k), dtype=bool)
    a, b = oracle.backward(cfg, h, w, gout), oracle.backward(cfg, h, w, gout, dropped=none)
    assert np.abs(a["dWr2"] - b["dWr2"]).max() > 1e-6
    # k = 1: the single survivor's gate is p / p = 1, a constant: the router gets no gradient
    cfg1, h1, w1, g1 = make_case(82, k=1)
    c = oracle.backward(cfg1, h1, w1, g1, dropped=np.zeros((cfg1.N, 1), dtype=bool))
    assert np.abs(c["dWr2"]).max() == 0.0 and np.abs(c["dWr1"]).max() == 0.0


def test_shuffled_slices_backward_is_the_permuted_backward():
    """Figure 5's shuffled layer is h' = P^-1 layer(P h) with a column permutation P, so its input
    gradient is P^-1 backward(P h, P gout) and the weight gradients are those of the inner layer.
    Checked by finite differences of the (separately pinned) shuffled forward."""
    cfg, h, w, gout = make_case(91, T=5, d=12, S=3)
    perm = np.random.default_rng(3).permutation(cfg.d)
    idx = oracle.forward_shuffled(cfg, h, w, perm)["topk_idx"]
    inner = oracle.backward(cfg, oracle.permute_columns(h, perm), w, oracle.permute_columns(gout, perm),
                            forced_idx=idx)
    dh = oracle.permute_columns(inner["dh"], perm, inverse=True)

    def loss(hh, ww):
        return float((oracle.forward_shuffled(cfg, hh, ww, perm, forced_idx=idx)["h_out"] * gout).sum())

    rng, eps = np.random.default_rng(4), 1e-5
    for _ in range(8):
        pos = (int(rng.integers(0, cfg.T)), int(rng.integers(0, cfg.d)))
        hi, lo = h.copy(), h.copy()
        hi[pos] += eps
        lo[pos] -= eps
        fd = (loss(hi, w) - loss(lo, w)) / (2 * eps)
        assert abs(fd - dh[pos]) <= 2e-6 * max(1.0, abs(fd)), (pos, fd, dh[pos])
    for name, g in (("W1", "dW1"), ("Wr1", "dWr1")):
        pos = tuple(int(rng.integers(0, s)) for s in w[name].shape)
        hi, lo = w[name].copy(), w[name].copy()
        hi[pos] += eps
        lo[pos] -= eps
        fd = (loss(h, {**w, name: hi}) - loss(h, {**w, name: lo})) / (2 * eps)
        assert abs(fd - inner[g][pos]) <= 2e-6 * max(1.0, abs(fd)), (name, pos)
