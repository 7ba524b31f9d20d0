"""Pins for the oracle's local update (Section 3 step (3)) and its bf16 wire cast. CPU only."""
import numpy as np
import torch

from oracle import oracle
from oracle.oracle import ADAM, BF16, F32, SGD, Oracle

f32 = np.float32


def _one_worker(n, opt, lr, theta, f64=False, **kw):
    return Oracle(W=1, n=n, packet_elems=8, p_grad=0.0, p_param=0.0, seed=0, grad_dtype=F32, replica_dtype=F32,
                  optimizer=opt, theta0=theta, lr=lr, f64=f64, **kw)


def test_sgd_constant_gradient_closed_form():
    n, T, lr = 64, 100, 1e-2
    rng = np.random.default_rng(0)
    theta = rng.standard_normal(n).astype(f32)
    g = rng.standard_normal(n).astype(f32)
    for f64 in (False, True):
        o = _one_worker(n, SGD, lr, theta, f64)
        for t in range(1, T + 1):
            o.step(t, [g])
        want = theta.astype(np.float64) - T * float(f32(lr)) * g.astype(np.float64)
        tol = 1e-12 if f64 else 2e-5
        assert np.max(np.abs(o.master - want)) <= tol * np.max(np.abs(want))


def test_adam_first_step_moves_by_lr_sign_g():
    n, lr = 256, 3e-4
    rng = np.random.default_rng(1)
    theta = rng.standard_normal(n).astype(f32)
    g = (rng.standard_normal(n) * 1e-3).astype(f32)
    o = _one_worker(n, ADAM, lr, theta, f64=True)
    o.step(1, [g])
    g64 = g.astype(np.float64)
    want = theta.astype(np.float64) - float(f32(lr)) * g64 / (np.abs(g64) + float(f32(1e-8)))
    assert np.allclose(o.master, want, rtol=1e-12, atol=0)
    big = np.abs(g64) > 1e-4                     # where eps is negligible the step is lr * sign(g)
    assert big.sum() > 100
    assert np.allclose((o.master - theta)[big], -float(f32(lr)) * np.sign(g64[big]), rtol=2e-4)


def test_adam_constant_gradient_closed_form():
    """With g constant, the bias-corrected moments are exactly g and g^2 at every step, so every
    step moves by lr * g / (|g| + eps)."""
    n, T, lr = 128, 50, 3e-4
    rng = np.random.default_rng(2)
    theta = rng.standard_normal(n).astype(f32)
    g = (rng.standard_normal(n) * 1e-3).astype(f32)
    g64 = g.astype(np.float64)
    want = theta.astype(np.float64) - T * float(f32(lr)) * g64 / (np.abs(g64) + float(f32(1e-8)))
    o = _one_worker(n, ADAM, lr, theta, f64=True)
    for t in range(1, T + 1):
        o.step(t, [g])
    assert np.max(np.abs(o.master - want)) <= 1e-9 * np.max(np.abs(want))
    o = _one_worker(n, ADAM, lr, theta)
    for t in range(1, T + 1):
        o.step(t, [g])
    assert np.max(np.abs(o.master - want)) <= 2e-6 * np.max(np.abs(want))


def test_adam_random_gradients_match_the_library_optimizer():
    n, T, lr = 512, 100, 3e-4
    rng = np.random.default_rng(3)
    theta = (rng.standard_normal(n) * 0.02).astype(f32)
    p = torch.nn.Parameter(torch.tensor(theta, dtype=torch.float64))
    b1, b2, eps = float(f32(0.9)), float(f32(0.95)), float(f32(1e-8))
    opt = torch.optim.Adam([p], lr=float(f32(lr)), betas=(b1, b2), eps=eps)
    o64 = _one_worker(n, ADAM, lr, theta, f64=True)
    o32 = _one_worker(n, ADAM, lr, theta)
    for t in range(1, T + 1):
        g = (rng.standard_normal(n) * 1e-3).astype(f32)
        p.grad = torch.tensor(g, dtype=torch.float64)
        opt.step()
        o64.step(t, [g])
        o32.step(t, [g])
    ref = p.detach().numpy()
    assert np.max(np.abs(o64.master - ref)) <= 1e-10 * np.max(np.abs(ref))
    moved = np.max(np.abs(ref - theta))
    assert np.max(np.abs(o32.master - ref)) <= 1e-5 * moved + 1e-7 * np.max(np.abs(ref))


def test_sgd_random_gradients_match_the_library_optimizer():
    n, T, lr = 512, 60, 1e-2
    rng = np.random.default_rng(4)
    theta = (rng.standard_normal(n) * 0.02).astype(f32)
    p = torch.nn.Parameter(torch.tensor(theta, dtype=torch.float64))
    opt = torch.optim.SGD([p], lr=float(f32(lr)))
    o = _one_worker(n, SGD, lr, theta, f64=True)
    for t in range(1, T + 1):
        g = (rng.standard_normal(n) * 1e-3).astype(f32)
        p.grad = torch.tensor(g, dtype=torch.float64)
        opt.step()
        o.step(t, [g])
    assert np.allclose(o.master, p.detach().numpy(), rtol=1e-13, atol=1e-18)


def test_learning_rate_can_change_between_steps():
    n = 16
    theta = np.ones(n, f32)
    g = np.ones(n, f32)
    o = _one_worker(n, SGD, 0.5, theta, f64=True)
    o.step(1, [g])
    o.set_lr(0.25)
    o.step(2, [g])
    assert np.all(o.master == 0.25)


def test_bf16_cast_is_round_to_nearest_even_like_the_library():
    rng = np.random.default_rng(5)
    x = np.concatenate([
        (rng.standard_normal(20000) * 0.02).astype(f32),
        (rng.standard_normal(2000) * 1e-30).astype(f32),
        np.array([0.0, -0.0, 1.0, -1.0, 3.3895314e38, 3.4e38, -3.4e38, 1e-45, 1.17549435e-38, np.inf, -np.inf],
                 dtype=f32),
        # exact ties: mantissa low half == 0x8000, with even and odd upper halves
        np.array([0x3F808000, 0x3F818000, 0xBF808000, 0xBF818000, 0x3F807FFF, 0x3F808001, 0x7F7F8000],
                 dtype=np.uint32).view(f32),
    ])
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = np.array([oracle.f32_to_bf16(float(v)) for v in x], dtype=np.uint16)
    assert np.array_equal(got, want)
    assert np.array_equal(oracle.cast_wire(x, BF16), want)            # the vectorised form used for large slabs
    assert oracle.f32_to_bf16(float("nan")) & 0x7FC0 == 0x7FC0       # NaN stays a (quiet) NaN
    back = oracle.bf16_bits_to_f32(want)
    assert np.array_equal(back.view(np.uint32), want.astype(np.uint32) << 16)
