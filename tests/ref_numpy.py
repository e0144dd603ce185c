"""A second, deliberately unfused statement of the Qwen3 forward pass in float64 numpy.

Written independently of the C oracle to pin it on small shapes: whole-sequence matrices, an explicit
[T][T] score matrix with an explicit causal mask, KV heads repeated explicitly for grouped-query attention,
angles computed from the closed form instead of a table.  Only the bf16 rounding of cached K and V is shared
in spirit (it is part of the definition of the path), and it is done here with torch's own cast.
"""
import numpy as np
import torch


def _f64(t):
    return t.to(torch.float64).numpy()


def _bf16_round(a):
    return torch.from_numpy(a).to(torch.float32).to(torch.bfloat16).to(torch.float64).numpy()


def rmsnorm(x, g, eps):
    return x / np.sqrt((x * x).mean(axis=-1, keepdims=True) + eps) * g


def rope(x, pos, theta):
    """x [..., T, d], pos [T]; half-split pairing."""
    d = x.shape[-1]
    i = np.arange(d // 2)
    ang = pos[:, None].astype(np.float64) * theta ** (-2.0 * i / d)[None, :]
    # the path stores cos/sin as fp32
    c = np.cos(ang).astype(np.float32).astype(np.float64)
    s = np.sin(ang).astype(np.float32).astype(np.float64)
    x1, x2 = x[..., : d // 2], x[..., d // 2:]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


def forward(shape, w, tokens, past_k=None, past_v=None):
    """Full-sequence forward.  past_k/past_v: optional per-layer lists of float64 [nkv][P][d] cache contents
    that precede `tokens`.  Returns (logits [T][V], taps [L+1][T][H], new_k, new_v per layer as stored)."""
    s = shape
    T = len(tokens)
    P = 0 if past_k is None else past_k[0].shape[1]
    d, nq, nkv = s.head_dim, s.n_q_heads, s.n_kv_heads
    G = nq // nkv
    x = _f64(w["embed"])[np.asarray(tokens)]
    taps = [x.copy()]
    pos = np.arange(P, P + T)
    ks, vs = [], []
    for l, lw in enumerate(w["layers"]):
        h = rmsnorm(x, _f64(lw["g_in"]), s.rms_eps)
        q = (h @ _f64(lw["wq"]).T).reshape(T, nq, d).transpose(1, 0, 2)
        k = (h @ _f64(lw["wk"]).T).reshape(T, nkv, d).transpose(1, 0, 2)
        v = (h @ _f64(lw["wv"]).T).reshape(T, nkv, d).transpose(1, 0, 2)
        q = rope(rmsnorm(q, _f64(lw["g_q"]), s.rms_eps), pos, s.rope_theta)
        k = rope(rmsnorm(k, _f64(lw["g_k"]), s.rms_eps), pos, s.rope_theta)
        k, v = _bf16_round(k), _bf16_round(v)
        if P:
            k = np.concatenate([past_k[l], k], axis=1)
            v = np.concatenate([past_v[l], v], axis=1)
        ks.append(k)
        vs.append(v)
        k_rep = np.repeat(k, G, axis=0)                       # [nq][P+T][d]
        v_rep = np.repeat(v, G, axis=0)
        scores = q @ k_rep.transpose(0, 2, 1) / np.sqrt(d)     # [nq][T][P+T]
        mask = np.arange(P + T)[None, :] > (pos[:, None])      # key position after the query's: hidden
        scores = np.where(mask[None], -np.inf, scores)
        scores = scores - scores.max(axis=-1, keepdims=True)
        pr = np.exp(scores)
        pr = pr / pr.sum(axis=-1, keepdims=True)
        o = (pr @ v_rep).transpose(1, 0, 2).reshape(T, nq * d)
        x = x + o @ _f64(lw["wo"]).T
        h = rmsnorm(x, _f64(lw["g_post"]), s.rms_eps)
        gate = h @ _f64(lw["w_gate"]).T
        up = h @ _f64(lw["w_up"]).T
        x = x + ((gate / (1.0 + np.exp(-gate))) * up) @ _f64(lw["w_down"]).T
        taps.append(x.copy())
    lm = w["embed"] if w.get("lm_head") is None else w["lm_head"]
    logits = rmsnorm(x, _f64(w["g_final"]), s.rms_eps) @ _f64(lm).T
    return logits, np.stack(taps), ks, vs
