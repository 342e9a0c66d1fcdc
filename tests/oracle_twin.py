"""A dense float64 re-evaluation of the operator used ONLY to pin the oracle on tiny shapes.

Written along a different route from the oracle: every quantised tensor is first
expanded to a dense float64 matrix (codes decoded through torch's float8 cast,
block scales broadcast element-wise), then the projections are plain matmuls.
Routing uses a stable lexicographic sort.  No blocking by scale group appears here.
"""
import numpy as np
import torch

_LUT = torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).to(torch.float64).numpy()


def bf16_bits_to_f64(bits):
    return torch.from_numpy(np.ascontiguousarray(bits, np.uint16).view(np.int16)).view(torch.bfloat16).to(torch.float64).numpy()


def dequant_blocks(q, s, group):
    return _LUT[q] * np.repeat(np.repeat(s.astype(np.float64), group, axis=-2), group, axis=-1)


def torch_quant(x32, group):
    v = torch.from_numpy(np.ascontiguousarray(x32, np.float32)).view(-1, group)
    sc = v.abs().amax(dim=1).clamp_min(1e-10) / 448.0
    q = (v / sc[:, None]).clamp(-448, 448).to(torch.float8_e4m3fn).view(torch.uint8)
    return q.numpy().reshape(x32.shape), sc.numpy().reshape(x32.shape[:-1] + (x32.shape[-1] // group,))


def route(hidden_bits, Wr_bits, bias, K, scoring, renorm, routed_scale=1.0):
    X, W = bf16_bits_to_f64(hidden_bits), bf16_bits_to_f64(Wr_bits)
    L = X @ W.T
    if scoring == 0:
        P = np.exp(L - L.max(axis=1, keepdims=True))
        V = P / P.sum(axis=1, keepdims=True)
        key = L
    else:
        V = 1.0 / (1.0 + np.exp(-L))
        key = V + (0.0 if bias is None else bias.astype(np.float64)[None, :])
    E = L.shape[1]
    ids = np.stack([np.lexsort((np.arange(E), -key[t]))[:K] for t in range(L.shape[0])]).astype(np.int32)
    v = np.take_along_axis(V, ids, axis=1)
    w = v / v.sum(axis=1, keepdims=True) if renorm else v
    return ids, (w * routed_scale).astype(np.float32), L


def forward(hidden_bits, Wr_bits, bias, W13q, W13s, W2q, W2s, K, scoring, renorm, group, routed_scale=1.0,
            ids=None, w=None):
    """Returns dict(ids, w, xq, xs, g [T,K,2I], act [T,K,I], hq, hs, y [T,K,H], out_f64 [T,H])."""
    if ids is None:
        ids, w, _ = route(hidden_bits, Wr_bits, bias, K, scoring, renorm, routed_scale)
    T, H = hidden_bits.shape
    I = W2q.shape[2]
    x32 = bf16_bits_to_f64(hidden_bits).astype(np.float32)
    xq, xs = torch_quant(x32, group)
    xd = _LUT[xq] * np.repeat(xs.astype(np.float64), group, axis=1)          # [T,H] dense
    W13 = dequant_blocks(W13q, W13s, group)                                   # [E,2I,H]
    W2 = dequant_blocks(W2q, W2s, group)                                      # [E,H,I]
    g = np.zeros((T, K, 2 * I)); act = np.zeros((T, K, I), np.float32)
    hq = np.zeros((T, K, I), np.uint8); hs = np.zeros((T, K, I // group), np.float32)
    y = np.zeros((T, K, H)); out = np.zeros((T, H))
    for t in range(T):
        for j in range(K):
            e = ids[t, j]
            g[t, j] = W13[e] @ xd[t]
            gate, up = g[t, j, :I], g[t, j, I:]
            act[t, j] = ((gate / (1.0 + np.exp(-gate))) * up).astype(np.float32)
            hq[t, j], hs[t, j] = torch_quant(act[t, j], group)
            hd = _LUT[hq[t, j]] * np.repeat(hs[t, j].astype(np.float64), group)
            y[t, j] = W2[e] @ hd
            out[t] += np.float64(w[t, j]) * y[t, j]
    return dict(ids=ids, w=w, xq=xq, xs=xs, g=g, act=act, hq=hq, hs=hs, y=y, out_f64=out)
