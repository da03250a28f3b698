"""CPU check of the tolerance that the tensor-mode policy is held to: a float64 / float16 emulation of that
mode's arithmetic, with the approximate tanh replaced by the exact one plus the worst perturbation its stated
error allows, must stay inside `logit_error_bound` for harness-like and for hostile weights."""
import numpy as np
import pytest

from paper_2207_07736_b200 import inputs
from tensor_bound import EPS_ACT, exact_logits64, logit_error_bound, split_params

TANH_ERR = 2.0 ** -10.987


def f16(x):
    return np.asarray(x, dtype=np.float64).astype(np.float16).astype(np.float64)


def emulate(p, obs, sign1, sign2):
    """Tensor-mode arithmetic with the tanh results of layer 1 / 2 pushed by sign1 / sign2 * TANH_ERR
    (each +1, -1 or an array of signs)."""
    W1, b1, W2, b2, W3, b3 = split_params(p)
    z1 = np.asarray(obs, dtype=np.float64) @ W1.T + b1                 # two-part operands: exact at this scale
    h1 = np.clip(np.tanh(f16(z1)) + sign1 * TANH_ERR, -1, 1)
    z2 = h1 @ f16(W2).T + b2
    h2 = np.clip(np.tanh(f16(z2)) + sign2 * TANH_ERR, -1, 1)
    return h2 @ W3.T + b3


def hostile_signs(p, obs):
    """The perturbation signs that push logit 0 up the most (first order)."""
    W1, b1, W2, b2, W3, b3 = split_params(p)
    h1 = np.tanh(np.asarray(obs, dtype=np.float64) @ W1.T + b1)
    slope2 = 1.0 - np.tanh(h1 @ W2.T + b2) ** 2                        # [M,64]
    return np.sign((W3[0] * slope2) @ W2), np.sign(W3[0])


@pytest.mark.parametrize("seed,bias,scale", [(1, 0.0, 1.0), (7, 0.3, 1.0), (3, 1.0, 4.0), (5, 0.0, 0.05)])
def test_bound_covers_the_emulated_tensor_mode(seed, bias, scale):
    rng = np.random.default_rng(seed)
    p = inputs.mlp_params(seed, bias).astype(np.float64)
    p[320:4416] *= scale                                               # hostile: large or tiny hidden weights
    obs = rng.uniform(-1, 1, (400, 4)) * np.array([2.4, 3, 0.21, 3])
    want, bound = exact_logits64(p, obs), logit_error_bound(p, obs)
    h1s, h2s = hostile_signs(p, obs)
    worst = 0.0
    for s1, s2 in ((+1.0, +1.0), (-1.0, -1.0), (rng.choice([-1.0, 1.0], size=(400, 64)), rng.choice([-1.0, 1.0], size=(400, 64))),
                   (h1s, h2s), (-h1s, -h2s)):
        err = np.abs(emulate(p, obs, s1, s2) - want)
        assert (err <= bound).all(), (float(err.max()), float(bound.min()))
        worst = max(worst, float((err / bound).max()))
    if scale <= 1.0:
        assert worst > 0.1                                             # the bound is not vacuous: hostile signs come close


def test_activation_error_model():
    """|tanh(f16(z)) - tanh(z)| <= 0.448 * 2^-11 for every z, so one activation is within EPS_ACT."""
    z = np.concatenate([np.linspace(-12, 12, 400001), np.random.default_rng(0).normal(0, 1, 200000)])
    assert np.abs(np.tanh(f16(z)) - np.tanh(z)).max() <= 0.448 * 2.0 ** -11
    assert EPS_ACT == TANH_ERR + 0.448 * 2.0 ** -11
