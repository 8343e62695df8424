"""Dense-mask attention written independently of the oracle (numpy, fp64).

Used only to pin the oracle.  RoPE is written as a complex multiplication
(x_a + i x_b) * exp(i theta), the mask is an explicit T x T matrix, and the
softmax is taken over whole rows with the mask added as -inf: none of this is
how the oracle is written.
"""
import numpy as np


def rope_complex(x, positions, base, interleaved=False, inv_freq=None):
    """x: [T, heads, d]; positions: [T] integers."""
    x = np.asarray(x, dtype=np.float64)
    T, heads, d = x.shape
    half = d // 2
    if inv_freq is None:
        inv_freq = base ** (-np.arange(half, dtype=np.float64) * 2.0 / d)
    ang = np.asarray(positions, dtype=np.float64)[:, None] * np.asarray(inv_freq)[None, :]
    rot = np.exp(1j * ang)[:, None, :]                      # [T,1,half]
    if interleaved:
        z = x[..., 0::2] + 1j * x[..., 1::2]
        z = z * rot
        y = np.empty_like(x)
        y[..., 0::2] = z.real
        y[..., 1::2] = z.imag
        return y
    z = x[..., :half] + 1j * x[..., half:]
    z = z * rot
    return np.concatenate([z.real, z.imag], axis=-1)


def causal_attention(q, k, v, base, scale=None, pos_offset=0, interleaved=False, inv_freq=None):
    """One monolithic causal pass over the whole sequence (the FULL condition).

    q [T,H,d], k,v [T,Hkv,d] before rotation.  Returns out [T,H,d], P [H,T,T].
    """
    q, k, v = (np.asarray(a, dtype=np.float64) for a in (q, k, v))
    T, H, d = q.shape
    Hkv = k.shape[1]
    G = H // Hkv
    scale = 1.0 / np.sqrt(d) if scale is None else scale
    pos = np.arange(T) + pos_offset
    qr = rope_complex(q, pos, base, interleaved, inv_freq)
    kr = rope_complex(k, pos, base, interleaved, inv_freq)
    mask = np.where(np.arange(T)[None, :] <= np.arange(T)[:, None], 0.0, -np.inf)   # [T,T]
    out = np.empty_like(q)
    probs = np.empty((H, T, T))
    for h in range(H):
        g = h // G
        s = (qr[:, h, :] @ kr[:, g, :].T) * scale + mask
        s = s - s.max(axis=1, keepdims=True)
        p = np.exp(s)
        p = p / p.sum(axis=1, keepdims=True)
        probs[h] = p
        out[:, h, :] = p @ v[:, g, :]
    return out, probs
