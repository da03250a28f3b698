"""Error bound of the tensor-mode (tolerance-mode) MLP policy, shared by the CPU check of the derivation and the
GPU tests.  One activation h = tanh~(f16(z)): the argument is rounded to FP16 (relative 2^-11; through tanh at
most 0.448 * 2^-11, the maximum of z / cosh(z)^2), then the approximate tanh adds at most 2^-10.987 (result in
FP16).  Layer-2 weights are rounded to FP16 (relative 2^-11); everything else carries 21 bits or more."""
import numpy as np

EPS_ACT = 2.0 ** -10.987 + 0.448 * 2.0 ** -11
EPS_F16 = 2.0 ** -11


def split_params(p):
    p = np.asarray(p, dtype=np.float64)
    return (p[0:256].reshape(64, 4), p[256:320], p[320:4416].reshape(64, 64), p[4416:4480],
            p[4480:4608].reshape(2, 64), p[4608:4610])


def exact_logits64(p, obs):
    W1, b1, W2, b2, W3, b3 = split_params(p)
    h1 = np.tanh(np.asarray(obs, dtype=np.float64) @ W1.T + b1)
    h2 = np.tanh(h1 @ W2.T + b2)
    return h2 @ W3.T + b3


def logit_error_bound(p, obs):
    """[M,2] bound on |tensor-mode logit - exact logit|, propagated through the layers in float64."""
    W1, b1, W2, b2, W3, b3 = split_params(p)
    h1 = np.tanh(np.asarray(obs, dtype=np.float64) @ W1.T + b1)                    # [M,64]
    e_z2 = (EPS_ACT + EPS_F16 * (np.abs(h1) + EPS_ACT)) @ np.abs(W2).T             # operand errors
    e_z2 += 80 * 2.0 ** -23 * (np.abs(h1) @ np.abs(W2).T + np.abs(b2))             # fp32 accumulation, split parts
    e_h2 = e_z2 + EPS_ACT                                                          # tanh is 1-Lipschitz
    return e_h2 @ np.abs(W3).T + 1e-5
