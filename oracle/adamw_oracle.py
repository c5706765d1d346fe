"""CPU fp64 oracle for the AdamW step applied to the parameters Muon does not
handle (RMSNorm gains, LM head, embeddings; Sec. 2.2 "Matching update RMS of
AdamW": learning rate and weight decay are shared with Muon).

TEST INFRASTRUCTURE ONLY; shares no code with the CUDA path.  The paper does
not restate AdamW; this follows the published algorithm (Adam with bias
correction, Kingma & Ba; decoupled weight decay, Loshchilov & Hutter):

    m_t = beta1 m_{t-1} + (1 - beta1) g
    v_t = beta2 v_{t-1} + (1 - beta2) g^2
    p_t = p_{t-1} - lr * ( (m_t / (1 - beta1^t)) / (sqrt(v_t / (1 - beta2^t)) + eps) + wd * p_{t-1} )

Pinned by closed forms in tests/test_adamw_oracle_pins.py (first step, constant
gradient, zero gradient, hand-computed scalars).
"""

from __future__ import annotations

import math

import numpy as np


def adamw_step(p, g, m, v, step, lr, wd, beta1=0.9, beta2=0.95, eps=1e-8):
    """One AdamW step; `step` counts from 1.  float64 arrays in, (p, m, v) out."""
    for x in (p, g, m, v):
        if np.asarray(x).dtype != np.float64:
            raise TypeError("oracle inputs must already be widened to float64")
    if step < 1:
        raise ValueError("step counts from 1")
    m_new = beta1 * m + (1.0 - beta1) * g
    v_new = beta2 * v + (1.0 - beta2) * g * g
    m_hat = m_new / (1.0 - math.pow(beta1, step))
    v_hat = v_new / (1.0 - math.pow(beta2, step))
    p_new = p - lr * (m_hat / (np.sqrt(v_hat) + eps) + wd * p)
    return p_new, m_new, v_new
