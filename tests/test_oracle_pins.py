"""Pins for the fp64 oracle: things the paper and the mathematics fix.

None of these call the oracle to check the oracle: the expected values come
from dense-mask brute force written differently (tests/bruteforce.py), from
closed forms, or from numbers the paper prints.
"""
import os

import numpy as np
import pytest

import oracle
from tests import bruteforce as bf

RNG = np.random.default_rng


def _qkv(rng, T, H, Hkv, d, scale=1.0):
    return (rng.standard_normal((T, H, d)) * scale,
            rng.standard_normal((T, Hkv, d)) * scale,
            rng.standard_normal((T, Hkv, d)) * scale)


def _fold(q, k, v, chunks, H, Hkv, d, base=10000.0, pos_shift=0, interleaved=False, **kw):
    c = oracle.OracleCache(H, Hkv, d, capacity=q.shape[0], rope_base=base,
                           interleaved=interleaved, **kw)
    outs, lens = [], []
    t0 = 0
    for n in chunks:
        outs.append(c.fold_step(q[t0:t0 + n], k[t0:t0 + n], v[t0:t0 + n], pos0=t0 + pos_shift))
        t0 += n
        lens.append(len(c))
    return np.concatenate(outs, axis=0), lens, c


# ---------------------------------------------------------------- brute force
@pytest.mark.parametrize("H,Hkv,d,T", [(1, 1, 2, 5), (4, 1, 8, 33), (4, 2, 8, 48), (6, 3, 16, 64)])
@pytest.mark.parametrize("interleaved", [False, True])
def test_single_step_matches_dense_mask_bruteforce(H, Hkv, d, T, interleaved):
    q, k, v = _qkv(RNG(1), T, H, Hkv, d)
    ref, _ = bf.causal_attention(q, k, v, 10000.0, interleaved=interleaved)
    got, _, _ = _fold(q, k, v, [T], H, Hkv, d, interleaved=interleaved)
    assert np.abs(got - ref).max() <= 1e-12


def test_rope_matches_complex_rotation():
    rng = RNG(2)
    x = rng.standard_normal((7, 3, 16))
    tab = oracle.inv_freq(500000.0, 16)
    assert np.allclose(tab, 500000.0 ** (-np.arange(8) * 2.0 / 16), rtol=1e-15, atol=0)
    for inter in (False, True):
        got = oracle.rope_fp64(x, 1000, tab, interleaved=inter)
        ref = bf.rope_complex(x, np.arange(7) + 1000, 500000.0, interleaved=inter)
        assert np.abs(got - ref).max() <= 1e-12


def test_custom_inv_freq_table_is_honoured():
    rng = RNG(3)
    T, H, Hkv, d = 24, 2, 1, 8
    q, k, v = _qkv(rng, T, H, Hkv, d)
    tab = np.array([1.0, 0.3, 0.01, 0.0007])
    ref, _ = bf.causal_attention(q, k, v, None, inv_freq=tab)
    got, _, _ = _fold(q, k, v, [10, 14], H, Hkv, d, inv_freq_table=tab)
    assert np.abs(got - ref).max() <= 1e-12


# ------------------------------------------------- the paper's defining invariant
def test_fold_equals_one_causal_pass_for_every_chunk_size():
    """Folding chunk by chunk == the FULL condition's single causal pass (Section 2)."""
    T, H, Hkv, d = 48, 4, 2, 8
    q, k, v = _qkv(RNG(4), T, H, Hkv, d)
    ref, _ = bf.causal_attention(q, k, v, 10000.0)
    for C in range(1, T + 1):
        chunks = [C] * (T // C) + ([T % C] if T % C else [])
        got, lens, _ = _fold(q, k, v, chunks, H, Hkv, d)
        assert np.abs(got - ref).max() <= 1e-12, C
        assert lens == list(np.cumsum(chunks))


def test_fold_with_mixed_chunk_lengths():
    T, H, Hkv, d = 64, 4, 1, 16
    q, k, v = _qkv(RNG(5), T, H, Hkv, d)
    ref, _ = bf.causal_attention(q, k, v, 10000.0)
    got, lens, _ = _fold(q, k, v, [17, 1, 1, 30, 8, 7], H, Hkv, d)
    assert np.abs(got - ref).max() <= 1e-12
    assert lens[-1] == T


def test_tiny_config_fold_equals_monolithic():
    """Config 1: 4 q heads / 1 KV head, d=64, C=64, 8 steps."""
    T, H, Hkv, d, C = 512, 4, 1, 64, 64
    q, k, v = _qkv(RNG(6), T, H, Hkv, d)
    ref, _ = bf.causal_attention(q, k, v, 10000.0)
    got, lens, _ = _fold(q, k, v, [C] * 8, H, Hkv, d)
    assert np.abs(got - ref).max() <= 1e-12
    assert lens == [C * (t + 1) for t in range(8)]      # len after t steps = t*C


def test_isolated_condition_is_a_step_on_an_empty_cache():
    T, H, Hkv, d = 16, 2, 2, 8
    q, k, v = _qkv(RNG(7), T, H, Hkv, d)
    c = oracle.OracleCache(H, Hkv, d, capacity=64)
    c.fold_step(q, k, v)
    c.reset()
    assert len(c) == 0
    got = c.fold_step(q, k, v, pos0=5)
    ref, _ = bf.causal_attention(q, k, v, 10000.0, pos_offset=5)
    assert np.abs(got - ref).max() <= 1e-12


# ----------------------------------------------------------------- softmax facts
def test_rows_sum_to_one_and_output_is_a_convex_combination():
    T, H, Hkv, d = 96, 4, 2, 8
    q, k, v = _qkv(RNG(8), T, H, Hkv, d, scale=3.0)
    c = oracle.OracleCache(H, Hkv, d, capacity=T)
    t0 = 0
    for n in (32, 32, 32):
        out, lse, rowsum = c.fold_step(q[t0:t0 + n], k[t0:t0 + n], v[t0:t0 + n], want_stats=True)
        assert np.abs(rowsum - 1.0).max() <= 1e-14
        assert np.isfinite(lse).all()
        for i in range(n):
            for h in range(H):
                vis = v[:t0 + i + 1, h // 2, :]
                assert (out[i, h] <= vis.max(axis=0) + 1e-12).all()
                assert (out[i, h] >= vis.min(axis=0) - 1e-12).all()
        t0 += n


def test_lse_matches_bruteforce_logsumexp():
    T, H, Hkv, d = 20, 2, 1, 8
    q, k, v = _qkv(RNG(9), T, H, Hkv, d)
    c = oracle.OracleCache(H, Hkv, d, capacity=T)
    _, lse, _ = c.fold_step(q, k, v, want_stats=True)
    qr = bf.rope_complex(q, np.arange(T), 10000.0)
    kr = bf.rope_complex(k, np.arange(T), 10000.0)
    for h in range(H):
        s = (qr[:, h] @ kr[:, 0].T) / np.sqrt(d)
        for i in range(T):
            assert abs(lse[i, h] - np.log(np.exp(s[i, :i + 1]).sum())) <= 1e-12


# ------------------------------------------------------------------ closed forms
def test_first_token_returns_its_own_value_row():
    q, k, v = _qkv(RNG(10), 8, 4, 2, 8)
    out, _, _ = _fold(q, k, v, [8], 4, 2, 8)
    for h in range(4):
        assert np.array_equal(out[0, h], v[0, h // 2])


def test_constant_value_rows_give_that_row():
    rng = RNG(11)
    q, k, _ = _qkv(rng, 40, 4, 2, 8)
    row = rng.standard_normal((2, 8))
    v = np.broadcast_to(row, (40, 2, 8)).copy()
    out, _, _ = _fold(q, k, v, [16, 24], 4, 2, 8)
    for h in range(4):
        assert np.abs(out[:, h] - row[h // 2]).max() <= 1e-13


def test_zero_queries_give_running_mean_of_values():
    rng = RNG(12)
    _, k, v = _qkv(rng, 50, 2, 1, 8)
    q = np.zeros((50, 2, 8))
    out, _, _ = _fold(q, k, v, [20, 30], 2, 1, 8)
    mean = np.cumsum(v[:, 0], axis=0) / np.arange(1, 51)[:, None]
    for h in range(2):
        assert np.abs(out[:, h] - mean).max() <= 1e-13


def test_position_zero_is_identity_and_rotation_keeps_pair_norms():
    rng = RNG(13)
    x = rng.standard_normal((1, 3, 16))
    tab = oracle.inv_freq(10000.0, 16)
    assert np.array_equal(oracle.rope_fp64(x, 0, tab), x)
    y = oracle.rope_fp64(np.repeat(x, 9, axis=0), 12345, tab)
    n_in = x[..., :8] ** 2 + x[..., 8:] ** 2
    n_out = y[..., :8] ** 2 + y[..., 8:] ** 2
    assert np.abs(n_out - n_in).max() <= 1e-12


def test_shifting_all_positions_leaves_outputs_unchanged():
    """RoPE scores depend on position differences only (continued positions, Section 2)."""
    T, H, Hkv, d = 40, 4, 2, 16
    q, k, v = _qkv(RNG(14), T, H, Hkv, d)
    a, _, _ = _fold(q, k, v, [10] * 4, H, Hkv, d, base=500000.0)
    b, _, _ = _fold(q, k, v, [10] * 4, H, Hkv, d, base=500000.0, pos_shift=100000)
    assert np.abs(a - b).max() <= 1e-9
    # and positions that do NOT continue across the boundary change the result
    c = oracle.OracleCache(H, Hkv, d, capacity=T, rope_base=500000.0)
    outs = [c.fold_step(q[t:t + 10], k[t:t + 10], v[t:t + 10], pos0=0) for t in range(0, T, 10)]
    assert np.abs(np.concatenate(outs) - a).max() > 1e-3


def test_gqa_equals_mha_with_replicated_kv_heads():
    T, H, Hkv, d = 24, 4, 2, 8
    q, k, v = _qkv(RNG(15), T, H, Hkv, d)
    a, _, _ = _fold(q, k, v, [8] * 3, H, Hkv, d)
    kk, vv = np.repeat(k, 2, axis=1), np.repeat(v, 2, axis=1)
    b, _, _ = _fold(q, kk, vv, [8] * 3, H, H, d)
    assert np.abs(a - b).max() <= 1e-14


def test_permuting_prefix_rows_leaves_outputs_unchanged():
    """Attention over the prefix is a set operation once keys carry their rotation."""
    rng = RNG(16)
    T, H, Hkv, d, P = 48, 2, 1, 8, 32
    q, k, v = _qkv(rng, T, H, Hkv, d)
    c1 = oracle.OracleCache(H, Hkv, d, capacity=T)
    c1.fold_step(q[:P], k[:P], v[:P])
    a = c1.fold_step(q[P:], k[P:], v[P:])
    # second cache: the same prefix, fed one token at a time in a permuted order,
    # each token at its ORIGINAL position
    perm = rng.permutation(P)
    c2 = oracle.OracleCache(H, Hkv, d, capacity=T)
    for r in perm:
        c2.fold_step(q[r:r + 1], k[r:r + 1], v[r:r + 1], pos0=int(r))
    b = c2.fold_step(q[P:], k[P:], v[P:], pos0=P)
    assert np.abs(a - b).max() <= 1e-12


def test_planted_key_is_recovered_through_a_deep_chain():
    """Kernel-level analogue of the needle test (Section 4): a key planted in chunk 0
    dominates a late query's row and the output approaches the planted value row."""
    rng = RNG(17)
    T, H, Hkv, d, C = 256, 2, 1, 16, 8
    q, k, v = _qkv(rng, T, H, Hkv, d, scale=0.1)
    tab = oracle.inv_freq(10000.0, d)
    needle_pos, query_pos = 3, T - 1
    direction = rng.standard_normal(d)
    direction /= np.linalg.norm(direction)
    # choose pre-rotation k, q whose ROTATED versions are aligned: rotate back by -pos
    def unrotate(vec, pos):
        ang = pos * tab
        z = (vec[:d // 2] + 1j * vec[d // 2:]) * np.exp(-1j * ang)
        return np.concatenate([z.real, z.imag])
    k[needle_pos, 0] = unrotate(direction * 30.0, needle_pos)
    q[query_pos, :] = unrotate(direction * 30.0, query_pos)
    out, lens, _ = _fold(q, k, v, [C] * (T // C), H, Hkv, d)
    assert lens[-1] == T
    for h in range(H):
        assert np.abs(out[query_pos, h] - v[needle_pos, 0]).max() <= 1e-9


# -------------------------------------------------------------- append / the cache
# ------------------------------------------------- sink + window variant
@pytest.mark.parametrize("n_sink,window,chunks", [
    (4, 12, [8] * 8), (4, 12, [5, 8, 1, 13, 7, 2, 16, 12]), (0, 9, [6] * 7), (3, 1, [4] * 6), (2, 40, [16] * 4),
])
def test_window_mode_equals_a_cache_that_is_literally_evicted_after_every_chunk(n_sink, window, chunks):
    """Section 6's StreamingLLM baseline: sinks plus a sliding window, eviction that leaves the kept
    rows at their positions.  The expected values come from a cache whose rows are deleted."""
    T, H, Hkv, d = sum(chunks), 4, 2, 8
    q, k, v = _qkv(RNG(31), T, H, Hkv, d)
    ref, held = bf.evicting_fold(q, k, v, chunks, n_sink, window, 10000.0)
    assert held <= n_sink + window                       # the cache capacity the paper quotes: 4 + 1020
    c = oracle.OracleCache(H, Hkv, d, capacity=T)
    c.set_window(n_sink, window)
    outs, t0 = [], 0
    for n in chunks:
        o, lse, rowsum = c.fold_step(q[t0:t0 + n], k[t0:t0 + n], v[t0:t0 + n], want_stats=True)
        assert np.abs(rowsum - 1.0).max() <= 1e-14
        outs.append(o)
        t0 += n
    assert np.abs(np.concatenate(outs) - ref).max() <= 1e-12


def test_window_that_covers_everything_is_the_plain_fold_and_a_far_key_is_lost_otherwise():
    T, H, Hkv, d, C = 96, 2, 1, 8, 8
    q, k, v = _qkv(RNG(32), T, H, Hkv, d)
    plain, _, _ = _fold(q, k, v, [C] * (T // C), H, Hkv, d)
    c = oracle.OracleCache(H, Hkv, d, capacity=T)
    c.set_window(0, T)
    wide = np.concatenate([c.fold_step(q[t:t + C], k[t:t + C], v[t:t + C]) for t in range(0, T, C)])
    assert np.array_equal(wide, plain)
    # a planted key outside sinks and window has no influence at all: changing its value row
    # changes nothing in the last chunk's output
    outs = []
    for bump in (0.0, 100.0):
        v2 = v.copy()
        v2[20] += bump                                   # row 20: not a sink, 68 rows before the last chunk
        c = oracle.OracleCache(H, Hkv, d, capacity=T)
        c.set_window(4, 16)
        for t in range(0, T, C):
            o = c.fold_step(q[t:t + C], k[t:t + C], v2[t:t + C])
        outs.append(o)
    assert np.array_equal(outs[0], outs[1])


# ------------------------------------------------- quantised storage (int8 round trip)
@pytest.mark.parametrize("bits,Q", [(8, 127), (4, 7)])
def test_int8_round_trip_is_round_to_nearest_on_a_grid_of_255_levels(bits, Q):
    """What 'symmetric intN per row, round to nearest' fixes without naming an implementation:
    integer codes within +-Q (127 for int8, 7 for int4), the largest element at +-Q, every stored value
    within half a grid step of the input (plus the bf16 rounding of the stored value), zero rows stay zero."""
    rng = RNG(41)
    x = (rng.standard_normal((64, 128)) * rng.uniform(0.01, 30.0, size=(64, 1))).astype(np.float32)
    x[7] = 0.0
    codes, scales, stored = oracle.quant_rows(x, bits)
    assert codes.dtype == np.int32 and np.abs(codes).max() == Q and np.abs(codes).min() >= 0
    assert len(np.unique(codes)) >= (15 if bits == 4 else 200)     # the grid is used, not a coarser one
    amax = np.abs(x).max(axis=1)
    big = np.abs(x).argmax(axis=1)
    rows = np.arange(64)
    assert np.array_equal(np.abs(codes[rows, big])[amax > 0], np.full((amax > 0).sum(), Q))
    assert np.array_equal(np.sign(codes[rows, big]), np.sign(x[rows, big]).astype(np.int32))
    assert np.allclose(scales, amax / float(Q), rtol=2e-7, atol=0)
    step = scales[:, None].astype(np.float64)
    exact = codes * step                                           # the grid point, before the bf16 rounding
    assert (np.abs(exact - x) <= 0.5 * step * (1 + 1e-5) + 1e-30).all()        # nearest: never more than half a step
    assert (np.abs(stored - exact) <= np.abs(exact) * 2.0 ** -8 + 1e-30).all()  # bf16: half an ulp of 8 bits
    assert not stored[7].any() and not codes[7].any() and scales[7] == 0.0
    # a truncating quantiser would be off by up to a whole step somewhere
    assert (np.abs(exact - x) > 0.25 * step).any()


@pytest.mark.parametrize("bits,Q", [(8, 127), (4, 7)])
def test_int8_round_trip_symmetries(bits, Q):
    rng = RNG(42)
    x = rng.standard_normal((16, 64)).astype(np.float32)
    c0, s0, y0 = oracle.quant_rows(x, bits)
    c1, s1, y1 = oracle.quant_rows(-x, bits)
    assert np.array_equal(c1, -c0) and np.array_equal(s1, s0) and np.array_equal(y1, -y0)
    c2, s2, y2 = oracle.quant_rows(x * np.float32(2.0 ** -5), bits)      # a power of two moves the scale only
    assert np.array_equal(c2, c0) and np.array_equal(s2, s0 * np.float32(2.0 ** -5)) and np.array_equal(y2, y0 * np.float32(2.0 ** -5))
    ints = rng.integers(-Q, Q + 1, size=(8, 32)).astype(np.float32)
    ints[:, 0] = float(Q)
    c3, s3, y3 = oracle.quant_rows(ints, bits)                           # rows already on the grid come back as they are
    assert np.array_equal(c3, ints.astype(np.int32)) and np.all(s3 == 1.0) and np.array_equal(y3, ints)


@pytest.mark.parametrize("bits,lo,hi", [(8, 1e-4, 3e-2), (4, 2e-2, 0.5)])
def test_quantised_fold_is_the_plain_fold_on_rows_that_went_through_the_round_trip(bits, lo, hi):
    """The cache of the quantised oracle, fed to a brute-force causal pass as already-rotated keys,
    reproduces its outputs; and against the unquantised fold the outputs move by a few per cent at
    most (noise-like perturbation, the paper's Discussion)."""
    T, H, Hkv, d, C = 96, 4, 2, 16, 16
    q, k, v = _qkv(RNG(43), T, H, Hkv, d)
    q, k, v = (a.astype(np.float32).astype(np.float64) for a in (q, k, v))
    plain, _, _ = _fold(q, k, v, [C] * (T // C), H, Hkv, d)
    c = oracle.OracleCache(H, Hkv, d, capacity=T)
    c.set_quant(bits)
    outs = [c.fold_step(q[t:t + C], k[t:t + C], v[t:t + C]) for t in range(0, T, C)]
    got = np.concatenate(outs)
    # stored keys = round trip of the fp32 rotation, stored values = round trip of v
    tab = oracle.inv_freq(10000.0, d)
    rot = oracle.rope_faithful(k.astype(np.float32), 0, tab)
    _, _, k_st = oracle.quant_rows(rot, bits)
    _, _, v_st = oracle.quant_rows(v.astype(np.float32), bits)
    assert np.array_equal(c.k(), np.transpose(k_st, (1, 0, 2)).astype(np.float64))
    assert np.array_equal(c.v(), np.transpose(v_st, (1, 0, 2)).astype(np.float64))
    qr = bf.rope_complex(q, np.arange(T), 10000.0)
    G = H // Hkv
    ref = np.empty_like(got)
    for h in range(H):
        s = (qr[:, h] @ k_st[:, h // G].astype(np.float64).T) / np.sqrt(d)
        s = np.where(np.arange(T)[None, :] <= np.arange(T)[:, None], s, -np.inf)
        p = np.exp(s - s.max(axis=1, keepdims=True))
        ref[:, h] = (p / p.sum(axis=1, keepdims=True)) @ v_st[:, h // G].astype(np.float64)
    assert np.abs(got - ref).max() <= 1e-12
    rel = np.sqrt(((got - plain) ** 2).sum() / (plain ** 2).sum())
    assert lo < rel < hi, rel                                 # int4 moves the outputs an order of magnitude more


def test_append_only_prefix_rows_are_bit_unchanged():
    T, H, Hkv, d = 30, 2, 2, 8
    q, k, v = _qkv(RNG(18), T, H, Hkv, d)
    c = oracle.OracleCache(H, Hkv, d, capacity=T)
    c.fold_step(q[:12], k[:12], v[:12])
    k_before, v_before = c.k().copy(), c.v().copy()
    c.fold_step(q[12:], k[12:], v[12:])
    assert np.array_equal(c.k()[:, :12], k_before)
    assert np.array_equal(c.v()[:, :12], v_before)
    # values are cached as given, keys after rotation at their own positions
    assert np.array_equal(c.v(), np.transpose(v, (1, 0, 2)))
    kr = bf.rope_complex(k, np.arange(T), 10000.0)
    assert np.abs(c.k() - np.transpose(kr, (1, 0, 2))).max() <= 1e-12


def test_capacity_overflow_changes_nothing():
    q, k, v = _qkv(RNG(19), 10, 2, 1, 8)
    c = oracle.OracleCache(2, 1, 8, capacity=12)
    c.fold_step(q, k, v)
    with pytest.raises(OverflowError):
        c.fold_step(q, k, v)
    assert len(c) == 10


def test_sampled_rows_equal_full_evaluation():
    q, k, v = _qkv(RNG(20), 24, 4, 2, 8)
    c1 = oracle.OracleCache(4, 2, 8, capacity=48)
    c2 = oracle.OracleCache(4, 2, 8, capacity=48)
    c1.fold_step(q, k, v)
    c2.fold_step(q, k, v, rows=[0])
    full = c1.fold_step(q, k, v)
    part = c2.fold_step(q, k, v, rows=[0, 7, 23])
    assert np.array_equal(part, full[[0, 7, 23]])
    assert len(c1) == len(c2) == 48


def test_cache_bytes_match_the_paper_s_printed_sizes():
    """Section 5: 32 layers x 8 KV heads x 128 x (K,V) x 2 B per token, and the table's GB."""
    per_token_all_layers = 32 * oracle.cache_bytes(8, 128, 1, 2)
    assert per_token_all_layers == 131072
    path = os.path.join(os.path.dirname(__file__), "golden", "cache_accounting.txt")
    rows = [l.split() for l in open(path) if l.strip() and not l.startswith("#")]
    assert len(rows) == 4
    for tokens, depth, gb in rows:
        tokens, depth, gb = int(tokens), int(depth), float(gb)
        total = 32 * oracle.cache_bytes(8, 128, tokens, 2)
        assert abs(total / 1e9 - gb) <= 0.005 + 1e-9          # printed to 2 decimals
        assert tokens // 256 - 1 == depth                   # chain depth at C = 256
    assert 32 * oracle.cache_bytes(8, 128, 131072, 2) == 17179869184


# ------------------------------------------------------- dtype-faithful rotation
def _bf16_round(x32):
    u = x32.astype(np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32)


@pytest.mark.parametrize("interleaved", [False, True])
def test_faithful_rotation_is_within_half_ulp_of_fp64(interleaved):
    rng = RNG(21)
    x = rng.standard_normal((64, 3, 32)).astype(np.float32)
    tab = oracle.inv_freq(500000.0, 32)
    exact = oracle.rope_fp64(x.astype(np.float64), 100000, tab, interleaved=interleaved)
    y32 = oracle.rope_faithful(x, 100000, tab, interleaved=interleaved, to_bf16=False)
    # three fp32 roundings (table value, cross product, fma): a few fp32 ulps of |x|
    scale = np.abs(x).max()
    assert np.abs(y32.astype(np.float64) - exact).max() <= 4 * 2.0 ** -24 * scale * 2
    y16 = oracle.rope_faithful(x, 100000, tab, interleaved=interleaved, to_bf16=True)
    # bf16 pattern: low 16 bits clear, and equal to RNE of the fp32 result
    assert (y16.view(np.uint32) & 0xFFFF == 0).all()
    assert np.array_equal(y16, _bf16_round(y32))
    ulp = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(exact), 1e-30))) - 7)
    assert (np.abs(y16.astype(np.float64) - exact) <= 0.5 * ulp + 1e-6).all()


def test_faithful_rotation_at_position_zero_is_identity():
    x = RNG(22).standard_normal((1, 2, 16)).astype(np.float32)
    tab = oracle.inv_freq(10000.0, 16)
    assert np.array_equal(oracle.rope_faithful(x, 0, tab), x)
