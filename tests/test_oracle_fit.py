"""Pins of the draft-head fitting oracle (paper Sec. II-A: cross-entropy of head i times lambda^i, base model
frozen): the analytic gradients against central finite differences of the loss, the loss against closed forms,
a one-parameter Adam trajectory worked out by hand, and the descent of the loss on a learnable toy stream."""
import numpy as np

from oracle import fit as F


def _problem(seed, T=7, d=5, V=6, heads=3):
    rng = np.random.default_rng(seed)
    W = rng.normal(0, 0.5, (heads, d, d)); b = rng.normal(0, 0.5, (heads, d)); U = rng.normal(0, 0.5, (heads, V, d))
    h = rng.normal(0, 1.0, (T, d))
    tg = rng.integers(0, V, (T, heads))
    for i in range(heads):
        tg[T - 1 - i:, i] = -1                                          # the last positions have no later token
    return W, b, U, h, tg


def test_gradients_match_finite_differences():
    W, b, U, h, tg = _problem(1)
    lam = 0.8
    loss, per, dW, db, dU = F.heads_grads(W, b, U, h, tg, lam)
    assert abs(loss - F.heads_loss(W, b, U, h, tg, lam)[0]) < 1e-12
    eps = 1e-6
    rng = np.random.default_rng(2)
    for arr, grad in ((W, dW), (b, db), (U, dU)):
        for _ in range(25):
            idx = tuple(int(rng.integers(0, s)) for s in arr.shape)
            old = arr[idx]
            arr[idx] = old + eps; lp = F.heads_loss(W, b, U, h, tg, lam)[0]
            arr[idx] = old - eps; lm = F.heads_loss(W, b, U, h, tg, lam)[0]
            arr[idx] = old
            assert abs((lp - lm) / (2 * eps) - grad[idx]) < 1e-7, (idx, (lp - lm) / (2 * eps), grad[idx])


def test_loss_closed_forms():
    W, b, U, h, tg = _problem(3, heads=2)
    # zero vocabulary matrices: every head predicts the uniform distribution, cross-entropy log V
    per = F.heads_loss(W, b, np.zeros_like(U), h, tg, 0.8)[1]
    assert np.allclose(per, np.log(U.shape[1]))
    # the weight of head i is lambda^i with i counted from 1 (Sec. II-A)
    total, per = F.heads_loss(W, b, U, h, tg, 0.5)
    assert abs(total - (0.5 * per[0] + 0.25 * per[1])) < 1e-12
    # a position without a target does not enter: dropping it from the stream changes nothing for that head
    t2 = tg.copy(); t2[0, 0] = -1
    per2 = F.heads_loss(W, b, U, h, t2, 0.5)[1]
    per3 = F.heads_loss(W, b, U, h[1:], tg[1:], 0.5)[1]
    assert abs(per2[0] - per3[0]) < 1e-12
    # z = h + SiLU(pre): with W = 0, b = 0 the block is the identity and the head is a softmax regression on h,
    # whose gradient with respect to U is (p - onehot)^T h / n
    W0, b0 = np.zeros_like(W), np.zeros_like(b)
    _, _, _, _, dU = F.heads_grads(W0, b0, U, h, tg, 1.0)
    lg = h @ U[0].T
    p = np.exp(lg - lg.max(1, keepdims=True)); p /= p.sum(1, keepdims=True)
    valid = tg[:, 0] >= 0
    p[valid, tg[valid, 0]] -= 1.0
    p[~valid] = 0
    assert np.allclose(dU[0], p.T @ h / valid.sum())


def test_silu_and_its_derivative():
    x = np.linspace(-6, 6, 41)
    assert np.allclose(F.silu(x), x / (1 + np.exp(-x)))
    e = 1e-6
    assert np.allclose(F.silu_grad(x), (F.silu(x + e) - F.silu(x - e)) / (2 * e), atol=1e-8)
    assert F.silu(0.0) == 0.0 and abs(F.silu_grad(0.0) - 0.5) < 1e-15


def test_adam_first_steps_by_hand_and_warmup():
    st = F.AdamState(np.zeros(1), np.zeros(1))
    p = np.array([1.0])
    # first step: m_hat = g, v_hat = g^2, so the move is lr * g / (|g| + eps) whatever the size of g
    p = F.adam_update(p, np.array([3.0]), st, 1, 0.1)
    assert abs(p[0] - (1.0 - 0.1 * 3.0 / (3.0 + 1e-8))) < 1e-15
    # second step with the same gradient: the bias-corrected moments are again g and g^2
    p2 = F.adam_update(p, np.array([3.0]), st, 2, 0.1)
    assert abs((p[0] - p2[0]) - 0.1 * 3.0 / (3.0 + 1e-8)) < 1e-12
    assert F.warmup_lr(1, 0.002, 40) == 0.002 / 40 and F.warmup_lr(40, 0.002, 40) == 0.002 and F.warmup_lr(400, 0.002, 40) == 0.002


def test_fitting_learns_a_deterministic_stream():
    """Hidden state = one-hot of the current token of a fixed cyclic stream: head i can learn token t+1+i exactly."""
    V, d, heads, T = 6, 6, 2, 60
    stream = np.arange(T + heads + 1) % V                           # a cycle: the next tokens are functions of the current one
    h = np.eye(V)[stream[:T]] * 3.0
    tg = np.stack([stream[2 + i:T + 2 + i] for i in range(heads)], axis=1)
    rng = np.random.default_rng(0)
    fit = F.HeadFitter(rng.normal(0, 0.02, (heads, d, d)), np.zeros((heads, d)), rng.normal(0, 0.02, (heads, V, d)), lr=0.05, warmup=5)
    first = fit.step(h, tg)[0]
    for _ in range(300):
        last, per = fit.step(h, tg)
    assert last < 0.05 * first and np.all(per < 0.1)
    z = h + F.silu(h @ fit.W[1].T + fit.b[1])
    assert np.array_equal((z @ fit.U[1].T).argmax(1), tg[:, 1])
