"""Single-query attention over the accessible tokens (oracle, test infrastructure).

Paper basis (Methodology, Preliminaries): for query head h of a layer with H_q
query heads and H_kv KV heads,
    a^h = softmax(q^h K_acc^T / sqrt(d)),   o^h = a^h V_acc,
where K_acc, V_acc are the keys and values that are currently accessible.
Query head h reads KV head floor(h / (H_q / H_kv)) (grouped-query attention).
Everything is float64; the caller rounds the output to the execution datatype.
"""

import numpy as np


def accessible_attention(q, k_acc, v_acc, scale):
    """q: [H_q, d]; k_acc, v_acc: [H_kv, n, d]; returns (out [H_q, d], probs [H_q, n])."""
    q = np.asarray(q, dtype=np.float64)
    k_acc = np.asarray(k_acc, dtype=np.float64)
    v_acc = np.asarray(v_acc, dtype=np.float64)
    n_q_heads, d = q.shape
    n_kv_heads, n, _ = k_acc.shape
    group = n_q_heads // n_kv_heads
    out = np.zeros((n_q_heads, d), dtype=np.float64)
    probs = np.zeros((n_q_heads, n), dtype=np.float64)
    if n == 0:
        return out, probs
    for h in range(n_q_heads):
        kv = h // group
        logits = (k_acc[kv] @ q[h]) * scale
        logits = logits - logits.max()
        e = np.exp(logits)
        p = e / e.sum()
        probs[h] = p
        out[h] = p @ v_acc[kv]
    return out, probs
