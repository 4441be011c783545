"""CPU oracle of the Mamba-based prompt classifier (test infrastructure only).

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this module; it shares nothing with
the CUDA library.  Section 2.4 and Section 3.3.3 describe the classifier as an embedding layer, a Mamba sequence
modelling layer, an adaptive pooling layer and a fully connected layer; the paper gives no formula and cites the Mamba
paper for the layer, so the layer below is that paper's block (selective state-space model, "S6"), step by step, in
float64, one token at a time:

    e_t   = E[token_t]                                            embedding row                     [D]
    u_t, z_t = split(W_in e_t)                                    input projection                  [Di], [Di]
    v_t   = silu(b_conv + sum_{j<Kc} w_conv[:, j] * u_{t-(Kc-1)+j})   causal depthwise convolution (zeros before the prompt)
    (r_t, B_t, C_t) = split(W_x v_t)                              input-dependent parameters        [R], [N], [N]
    dt_t  = softplus(W_dt r_t + b_dt)                             step size per channel             [Di]
    h_t   = exp(dt_t (x) A) * h_{t-1} + (dt_t * v_t) (x) B_t      A = -exp(A_log), h_{-1} = 0        [Di][N]
    y_t   = h_t C_t + D_skip * v_t                                                                   [Di]
    o_t   = W_out (y_t * silu(z_t))                               output projection                 [D]
    pooled = mean_t o_t                                           adaptive average pooling to one position
    scores = W_fc pooled + b_fc;  class = argmax (lowest index on ties)

Readings: the pooling is the average (the paper says "adaptive pooling" without the kind); the Mamba layer is the bare
block (no residual connection and no normalisation around a single layer); sizes are not given and are parameters.
"""
from __future__ import annotations

import numpy as np


def silu(x):
    return x / (1.0 + np.exp(-x))


def softplus(x):
    x = np.asarray(x, dtype=np.float64)
    return np.where(x > 30.0, x, np.log1p(np.exp(np.minimum(x, 30.0))))


def causal_depthwise_conv(u, w_conv, b_conv):
    """u [P][Di], w_conv [Di][Kc], b_conv [Di] -> [P][Di]; position t sees u_{t-Kc+1..t}, zeros before the start."""
    P, Di = u.shape
    Kc = w_conv.shape[1]
    out = np.zeros((P, Di))
    for t in range(P):
        acc = b_conv.astype(np.float64).copy()
        for j in range(Kc):
            s = t - (Kc - 1) + j
            if s >= 0:
                acc += w_conv[:, j] * u[s]
        out[t] = acc
    return out


def selective_scan(v, dt, A, B, C, D_skip):
    """v, dt [P][Di]; A [Di][N]; B, C [P][N]; D_skip [Di] -> y [P][Di], the recurrence one token at a time."""
    P, Di = v.shape
    h = np.zeros_like(A, dtype=np.float64)
    y = np.zeros((P, Di))
    for t in range(P):
        h = np.exp(dt[t][:, None] * A) * h + (dt[t] * v[t])[:, None] * B[t][None, :]
        y[t] = h @ C[t] + D_skip * v[t]
    return y


def forward(w, tokens):
    """Scores [n_classes] (float64), the pooled vector and the per-token outputs for one prompt.  w: dict of arrays
    embed [V][D], w_in [2Di][D], w_conv [Di][Kc], b_conv [Di], w_x [R+2N][Di], w_dt [Di][R], b_dt [Di], a_log [Di][N],
    d_skip [Di], w_out [D][Di], w_fc [K][D], b_fc [K]."""
    f = {k: np.asarray(a, dtype=np.float64) for k, a in w.items()}
    Di, R = f["w_dt"].shape
    N = f["a_log"].shape[1]
    e = f["embed"][np.asarray(tokens, dtype=np.int64)]
    uz = e @ f["w_in"].T
    u, z = uz[:, :Di], uz[:, Di:]
    v = silu(causal_depthwise_conv(u, f["w_conv"], f["b_conv"]))
    x_dbl = v @ f["w_x"].T
    r, B, C = x_dbl[:, :R], x_dbl[:, R:R + N], x_dbl[:, R + N:R + 2 * N]
    dt = softplus(r @ f["w_dt"].T + f["b_dt"])
    y = selective_scan(v, dt, -np.exp(f["a_log"]), B, C, f["d_skip"])
    o = (y * silu(z)) @ f["w_out"].T
    pooled = o.mean(axis=0)
    scores = f["w_fc"] @ pooled + f["b_fc"]
    return scores, pooled, o


def classify(w, tokens):
    scores, _, _ = forward(w, tokens)
    return int(np.argmax(scores)), scores
