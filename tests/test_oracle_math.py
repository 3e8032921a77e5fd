"""Pins for the checker's arithmetic: exp, softmax-CE / MSE gradients, L2 term, Adam.

Each check is against something the checker did not write itself: libm, torch autograd,
central finite differences, torch.optim.Adam, closed forms, and scikit-learn's own MLP
(the implementation the paper's Table 1 names as "MLP-adam").
"""
import math

import numpy as np
import pytest
import torch

import oracle


def unpack(theta, d, H, C):
    o = 0
    W1 = theta[o:o + d * H].reshape(d, H); o += d * H
    b1 = theta[o:o + H]; o += H
    W2 = theta[o:o + H * C].reshape(H, C); o += H * C
    b2 = theta[o:o + C]
    return W1, b1, W2, b2


def torch_loss(theta, xb, yb, d, H, C, task, alpha):
    """Independent statement of the minibatch loss with autograd-ready tensors."""
    W1, b1, W2, b2 = unpack(theta, d, H, C)
    z2 = torch.relu(xb @ W1 + b1) @ W2 + b2
    Bs = xb.shape[0]
    if task == 0:
        data = torch.nn.functional.cross_entropy(z2, yb.long(), reduction="mean")
    else:
        data = 0.5 * torch.mean((z2[:, 0] - yb) ** 2)
    return data + alpha / (2.0 * Bs) * ((W1 ** 2).sum() + (W2 ** 2).sum())


def test_exp_against_libm():
    xs = np.concatenate([np.linspace(-86.0, 0.0, 200001), -np.logspace(-8, 1.9, 5000),
                         np.linspace(0.0, 88.0, 20001)]).astype(np.float32)
    worst = 0.0
    for x in xs[::7]:
        got = oracle.expf(x)
        want = math.exp(float(x))
        ulp = np.spacing(np.float32(want))
        worst = max(worst, abs(got - want) / float(ulp))
    assert worst <= 2.0, worst
    assert oracle.expf(0.0) == 1.0
    assert oracle.expf(-87.0) == 0.0 and oracle.expf(-np.inf) == 0.0
    assert math.isnan(oracle.expf(float("nan")))
    ys = [oracle.expf(x) for x in np.linspace(-20, 0, 4001, dtype=np.float32)]
    assert all(b >= a for a, b in zip(ys, ys[1:]))


@pytest.mark.parametrize("task,C", [(0, 3), (0, 2), (1, 1)])
def test_gradient_matches_autograd_and_finite_differences(task, C):
    rng = np.random.default_rng(1)
    d, H, Bs, alpha = 3, 4, 5, 0.3
    P = oracle.param_count(d, H, C)
    theta = rng.normal(0, 0.7, P)
    xb = rng.normal(size=(Bs, d))
    yb = rng.integers(0, C, Bs).astype(np.float64) if task == 0 else rng.normal(size=Bs)
    loss, g = oracle.loss_grad(oracle.MODE_F64, d, H, C, task, alpha, theta, xb, yb)
    # (a) autograd
    th_t = torch.tensor(theta, dtype=torch.float64, requires_grad=True)
    lt = torch_loss(th_t, torch.tensor(xb), torch.tensor(yb), d, H, C, task, alpha)
    lt.backward()
    assert abs(loss - lt.item()) < 1e-12 * max(1.0, abs(loss))
    np.testing.assert_allclose(g, th_t.grad.numpy(), rtol=1e-10, atol=1e-12)
    # (b) central differences of the checker's own loss
    h = 1e-6
    fd = np.zeros(P)
    for i in range(P):
        tp, tm = theta.copy(), theta.copy()
        tp[i] += h; tm[i] -= h
        fd[i] = (oracle.loss_grad(1, d, H, C, task, alpha, tp, xb, yb)[0]
                 - oracle.loss_grad(1, d, H, C, task, alpha, tm, xb, yb)[0]) / (2 * h)
    np.testing.assert_allclose(g, fd, rtol=1e-6, atol=1e-8)
    # (c) float mode agrees with double mode to float accuracy
    th32 = theta.astype(np.float32).astype(np.float64)
    x32 = xb.astype(np.float32).astype(np.float64)
    y32 = yb.astype(np.float32).astype(np.float64)
    l32, g32 = oracle.loss_grad(oracle.MODE_F32, d, H, C, task, alpha, th32, x32, y32)
    l64, g64 = oracle.loss_grad(oracle.MODE_F64, d, H, C, task, alpha, th32, x32, y32)
    assert abs(l32 - l64) < 1e-5 * max(1.0, abs(l64))
    np.testing.assert_allclose(g32, g64, rtol=1e-4, atol=1e-6)


def test_gradient_wider_shapes_against_autograd():
    rng = np.random.default_rng(2)
    for (d, H, C, Bs, task) in [(30, 57, 2, 17, 0), (64, 50, 10, 33, 0), (10, 20, 1, 9, 1)]:
        P = oracle.param_count(d, H, C)
        theta = rng.normal(0, 0.3, P)
        xb = rng.normal(size=(Bs, d))
        yb = rng.integers(0, C, Bs).astype(np.float64) if task == 0 else rng.normal(size=Bs)
        loss, g = oracle.loss_grad(1, d, H, C, task, 0.01, theta, xb, yb)
        th_t = torch.tensor(theta, requires_grad=True)
        lt = torch_loss(th_t, torch.tensor(xb), torch.tensor(yb), d, H, C, task, 0.01)
        lt.backward()
        assert abs(loss - lt.item()) < 1e-11 * max(1.0, abs(loss))
        np.testing.assert_allclose(g, th_t.grad.numpy(), rtol=1e-9, atol=1e-12)


def test_l2_term_closed_form_and_alpha_zero():
    rng = np.random.default_rng(3)
    d, H, C, Bs = 4, 6, 3, 7
    P = oracle.param_count(d, H, C)
    theta = rng.normal(size=P)
    xb = rng.normal(size=(Bs, d)); yb = rng.integers(0, C, Bs).astype(float)
    l0, g0 = oracle.loss_grad(1, d, H, C, 0, 0.0, theta, xb, yb)
    la, ga = oracle.loss_grad(1, d, H, C, 0, 2.5, theta, xb, yb)
    W1, b1, W2, b2 = unpack(theta, d, H, C)
    sq = (W1 ** 2).sum() + (W2 ** 2).sum()
    assert abs((la - l0) - 2.5 / (2 * Bs) * sq) < 1e-12 * sq
    dW1, db1, dW2, db2 = unpack(ga - g0, d, H, C)
    np.testing.assert_allclose(dW1, 2.5 / Bs * W1, rtol=1e-12)
    np.testing.assert_allclose(dW2, 2.5 / Bs * W2, rtol=1e-12)
    assert np.all(db1 == 0) and np.all(db2 == 0)  # biases unpenalised


def test_softmax_properties():
    # the gradient wrt b2 is sum_b (p - onehot)/Bs: recover p and check it is a distribution,
    # shift invariant, and for C=2 the logistic of the logit difference
    d, H, C = 2, 3, 4
    P = oracle.param_count(d, H, C)
    rng = np.random.default_rng(4)
    theta = rng.normal(size=P).astype(np.float32).astype(np.float64)
    x = rng.normal(size=(1, d)).astype(np.float32).astype(np.float64)
    _, g = oracle.loss_grad(0, d, H, C, 0, 0.0, theta, x, np.array([1.0]))
    p = g[-C:].copy(); p[1] += 1.0
    assert abs(p.sum() - 1.0) < C * 1.2e-7 and np.all(p >= 0)
    th2 = theta.copy(); th2[-C:] += 8.0  # shift every logit by the same exactly-representable amount
    _, g2 = oracle.loss_grad(0, d, H, C, 0, 0.0, th2, x, np.array([1.0]))
    np.testing.assert_allclose(g2[-C:], g[-C:], rtol=0, atol=3e-7)
    C = 2
    P = oracle.param_count(d, H, C)
    theta = rng.normal(size=P)
    _, g = oracle.loss_grad(1, d, H, C, 0, 0.0, theta, x, np.array([0.0]))
    W1, b1, W2, b2 = unpack(theta, d, H, C)
    z = np.maximum(x @ W1 + b1, 0) @ W2 + b2
    assert abs(g[-1] - 1.0 / (1.0 + math.exp(-(z[0, 1] - z[0, 0])))) < 1e-12
    # loss at zero weights is ln C
    l, _ = oracle.loss_grad(1, d, H, C, 0, 0.0, np.zeros(P), x, np.array([0.0]))
    assert abs(l - math.log(2.0)) < 1e-15


def test_adam_first_step_closed_form_and_lr_zero():
    rng = np.random.default_rng(5)
    P = 50
    th = rng.normal(size=P); g = rng.normal(size=P) * 10.0 ** rng.uniform(-6, 2, P)
    lr, b1, b2, eps = 0.01, 0.9, 0.999, 1e-8
    t1, m1, v1 = oracle.adam_steps(1, th, np.zeros(P), np.zeros(P), g, lr, b1, b2, eps)
    want = th - lr * g / (np.abs(g) + eps / math.sqrt(1 - b2))
    np.testing.assert_allclose(t1, want, rtol=1e-12)
    np.testing.assert_allclose(m1, (1 - b1) * g, rtol=1e-15)
    np.testing.assert_allclose(v1, (1 - b2) * g * g, rtol=1e-15)
    # lr = 0 leaves the parameters bit-unchanged (both modes), whatever the gradients
    grads = rng.normal(size=(25, P))
    for mode in (0, 1):
        th0 = th.astype(np.float32).astype(np.float64)
        t, _, _ = oracle.adam_steps(mode, th0, np.zeros(P), np.zeros(P), grads, 0.0, b1, b2, eps)
        assert np.array_equal(t, th0)


def test_adam_matches_torch_optimizer_over_many_steps():
    # torch.optim.Adam applies eps to sqrt(v_hat); with a tiny eps both forms coincide
    rng = np.random.default_rng(6)
    P, S = 40, 60
    th = rng.normal(size=P)
    grads = rng.normal(size=(S, P)) * np.linspace(1.0, 0.1, S)[:, None]
    lr, b1, b2, eps = 0.003, 0.8, 0.97, 1e-14
    got, _, _ = oracle.adam_steps(1, th, np.zeros(P), np.zeros(P), grads, lr, b1, b2, eps)
    p = torch.tensor(th.copy(), requires_grad=True)
    opt = torch.optim.Adam([p], lr=lr, betas=(b1, b2), eps=eps)
    for s in range(S):
        p.grad = torch.tensor(grads[s].copy())
        opt.step()
    np.testing.assert_allclose(got, p.detach().numpy(), rtol=1e-9, atol=1e-12)
    # float mode tracks double mode
    g32 = grads.astype(np.float32).astype(np.float64)
    th32 = th.astype(np.float32).astype(np.float64)
    a, _, _ = oracle.adam_steps(0, th32, np.zeros(P), np.zeros(P), g32, lr, b1, b2, 1e-8)
    b, _, _ = oracle.adam_steps(1, th32, np.zeros(P), np.zeros(P), g32, lr, b1, b2, 1e-8)
    np.testing.assert_allclose(a, b, rtol=2e-5, atol=2e-6)


def test_adam_eps_scaling_matches_textbook_form():
    # Kingma & Ba Algorithm 1 with eps_hat_t = eps / sqrt(1 - beta2^t) is the same update
    rng = np.random.default_rng(7)
    P, S = 8, 12
    th = rng.normal(size=P); grads = rng.normal(size=(S, P))
    lr, b1, b2, eps = 0.05, 0.6, 0.9, 1e-3
    got, _, _ = oracle.adam_steps(1, th, np.zeros(P), np.zeros(P), grads, lr, b1, b2, eps)
    m = np.zeros(P); v = np.zeros(P); x = th.copy()
    for t in range(1, S + 1):
        g = grads[t - 1]
        m = b1 * m + (1 - b1) * g
        v = b2 * v + (1 - b2) * g * g
        mhat = m / (1 - b1 ** t); vhat = v / (1 - b2 ** t)
        x = x - lr * mhat / (np.sqrt(vhat) + eps / math.sqrt(1 - b2 ** t))
    np.testing.assert_allclose(got, x, rtol=1e-11)


def _sklearn_steps(task, C, n_steps):
    """Drive scikit-learn's MLP (adam solver) from given weights with full-batch steps."""
    sk = pytest.importorskip("sklearn.neural_network")
    rng = np.random.default_rng(8)
    n, d, H = 24, 5, 7
    X = rng.normal(size=(n, d))
    y = (np.arange(n) % C).astype(np.float64) if task == 0 else rng.normal(size=n)
    alpha, lr, b1, b2, eps = 0.37, 0.02, 0.85, 0.95, 1e-7
    kw = dict(hidden_layer_sizes=(H,), activation="relu", solver="adam", alpha=alpha, batch_size=n,
              learning_rate_init=lr, beta_1=b1, beta_2=b2, epsilon=eps, shuffle=False, random_state=0)
    est = sk.MLPClassifier(**kw) if task == 0 else sk.MLPRegressor(**kw)
    if task == 0:
        est.partial_fit(X, y.astype(int), classes=np.arange(C))
    else:
        est.partial_fit(X, y)
    opt = getattr(est, "_optimizer", None)
    if opt is None or not all(hasattr(opt, a) for a in ("ms", "vs", "t")):
        pytest.skip("scikit-learn internals differ from the expected layout")
    P = oracle.param_count(d, H, C)
    theta0 = rng.normal(0, 0.5, P)
    W1, c1, W2, c2 = unpack(theta0, d, H, C)
    est.coefs_[0][...] = W1; est.intercepts_[0][...] = c1
    est.coefs_[1][...] = W2; est.intercepts_[1][...] = c2
    for arr in list(opt.ms) + list(opt.vs):
        arr[...] = 0.0
    opt.t = 0
    for _ in range(n_steps):
        if task == 0:
            est.partial_fit(X, y.astype(int))
        else:
            est.partial_fit(X, y)
    sk_theta = np.concatenate([est.coefs_[0].ravel(), est.intercepts_[0], est.coefs_[1].ravel(),
                               est.intercepts_[1]])
    th = theta0.copy(); m = np.zeros(P); v = np.zeros(P)
    # the checker: same full-batch gradient, Adam state carried across calls
    grads = []
    for s in range(n_steps):
        # replay from scratch so that beta^t products restart at t=0 inside adam_steps
        th_s = theta0.copy(); m = np.zeros(P); v = np.zeros(P)
        if grads:
            th_s, m, v = oracle.adam_steps(1, th_s, m, v, np.array(grads), lr, b1, b2, eps)
        grads.append(oracle.loss_grad(1, d, H, C, task, alpha, th_s, X, y)[1])
    th, _, _ = oracle.adam_steps(1, theta0.copy(), np.zeros(P), np.zeros(P), np.array(grads), lr, b1, b2, eps)
    return th, sk_theta


def test_one_and_five_steps_match_scikit_learn_multiclass():
    for steps in (1, 5):
        ours, theirs = _sklearn_steps(0, 3, steps)
        np.testing.assert_allclose(ours, theirs, rtol=1e-9, atol=1e-11)


def test_five_steps_match_scikit_learn_regressor():
    ours, theirs = _sklearn_steps(1, 1, 5)
    np.testing.assert_allclose(ours, theirs, rtol=1e-9, atol=1e-11)
