"""Independent dense float64 decoder built from library routines (torch matmul, softmax, complex
multiply for the rotary embedding).  No cache: every call runs the full causal pass over all input
rows.  It exists only to pin the oracle's decoder; it shares nothing with oracle/ or the CUDA code."""
import math

import torch


def f64(t):
    return t.to(torch.float64)


def rmsnorm(x, g, eps):
    return x * torch.rsqrt((x * x).mean(-1, keepdim=True) + eps) * f64(g)


def rope(x, n_heads, theta):
    T, d = x.shape
    hd = d // n_heads
    xc = torch.view_as_complex(x.reshape(T, n_heads, hd // 2, 2).contiguous())
    freq = theta ** (-torch.arange(0, hd, 2, dtype=torch.float64) / hd)
    ang = torch.arange(T, dtype=torch.float64)[:, None] * freq[None, :]
    rot = torch.polar(torch.ones_like(ang), ang)
    return torch.view_as_real(xc * rot[:, None, :]).reshape(T, d)


def quant(x, kv_dtype):
    x = x.to(torch.float32)
    if kv_dtype == "bf16":
        x = x.to(torch.bfloat16)
    return x.to(torch.float64)


def dense_forward(weights, shape, X, kv_dtype="bf16", eps=1e-5, theta=10000.0):
    """X: float64 [T, d] input rows.  Returns (logits [T, V], residual-after-each-half-layer list)."""
    T, d = X.shape
    H = shape.n_heads
    hd = d // H
    mask = torch.full((T, T), float("-inf"), dtype=torch.float64).triu(1)
    trace = []
    h = X.clone()
    for l in range(shape.n_layers):
        a = rmsnorm(h, weights["attn_norm"][l], eps)
        q = rope(a @ f64(weights["wq"][l]).T, H, theta)
        k = quant(rope(a @ f64(weights["wk"][l]).T, H, theta), kv_dtype)
        v = quant(a @ f64(weights["wv"][l]).T, kv_dtype)
        qh, kh, vh = (t.reshape(T, H, hd).transpose(0, 1) for t in (q, k, v))
        att = torch.softmax(qh @ kh.transpose(1, 2) / math.sqrt(hd) + mask, dim=-1) @ vh
        h = h + att.transpose(0, 1).reshape(T, d) @ f64(weights["wo"][l]).T
        trace.append(h.clone())
        b = rmsnorm(h, weights["ffn_norm"][l], eps)
        g = b @ f64(weights["wgate"][l]).T
        u = torch.nn.functional.silu(g) * (b @ f64(weights["wup"][l]).T)
        h = h + u @ f64(weights["wdown"][l]).T
        trace.append(h.clone())
    logits = rmsnorm(h, weights["final_norm"], eps) @ f64(weights["lm_head"]).T
    return logits, trace
