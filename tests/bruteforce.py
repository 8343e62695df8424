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


def evicting_fold(q, k, v, chunks, n_sink, window, base, scale=None):
    """Chunk-by-chunk attention over a cache that is literally evicted after every chunk.

    The cache is a list of (rotated key, value) rows; a chunk attends to the rows the cache holds
    plus its own rows causally; afterwards the chunk's rows are appended and everything except the
    first n_sink rows ever appended and the last `window` rows is deleted.  Rows keep the rotation
    of the position they were appended at (no re-anchoring).  Returns out [T,H,d] and the largest
    number of rows the cache held after an eviction.
    """
    q, k, v = (np.asarray(a, dtype=np.float64) for a in (q, k, v))
    T, H, d = q.shape
    Hkv = k.shape[1]
    G = H // Hkv
    scale = 1.0 / np.sqrt(d) if scale is None else scale
    kept_k = [[] for _ in range(Hkv)]          # per KV head: list of rotated key rows
    kept_v = [[] for _ in range(Hkv)]
    kept_idx = []                              # which original rows the cache holds
    out = np.empty_like(q)
    held = 0
    t0 = 0
    for n in chunks:
        pos = np.arange(t0, t0 + n)
        qr = rope_complex(q[t0:t0 + n], pos, base)
        kr = rope_complex(k[t0:t0 + n], pos, base)
        for h in range(H):
            g = h // G
            for i in range(n):
                keys = np.array(kept_k[g] + [kr[j, g] for j in range(i + 1)])
                vals = np.array(kept_v[g] + [v[t0 + j, g] for j in range(i + 1)])
                s = keys @ qr[i, h] * scale
                p = np.exp(s - s.max())
                out[t0 + i, h] = (p / p.sum()) @ vals
        for g in range(Hkv):
            kept_k[g] += [kr[j, g] for j in range(n)]
            kept_v[g] += [v[t0 + j, g] for j in range(n)]
        kept_idx += list(range(t0, t0 + n))
        # eviction: the first n_sink rows ever seen stay, and the most recent `window`
        keep = [x for x, idx in enumerate(kept_idx) if idx < n_sink or idx >= t0 + n - window]
        for g in range(Hkv):
            kept_k[g] = [kept_k[g][x] for x in keep]
            kept_v[g] = [kept_v[g][x] for x in keep]
        kept_idx = [kept_idx[x] for x in keep]
        held = max(held, len(kept_idx))
        t0 += n
    return out, held
