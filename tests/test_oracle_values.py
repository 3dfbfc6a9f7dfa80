"""Pins for the oracle's values: brute force written here from Eq. 1-3, library routines,
closed forms and invariants.  No expectation below is produced by the oracle itself."""
import math

import numpy as np
import pytest
import scipy.special

import oracle
from paper_2012_01114_b200 import inputs


def brute_force(q, k, v, scale=1.0, masked=False):
    """Eq. 1-3 with pure-Python loops, literal form (no max subtraction).  For `masked`, the practice
    Sec. 5.1 describes: all n^2 weights are produced, then those above the diagonal are set to -inf."""
    n, d = len(q), len(q[0])
    wp = [[scale * sum(q[i][l] * k[j][l] for l in range(d)) for j in range(n)] for i in range(n)]
    if masked:
        for i in range(n):
            for j in range(i + 1, n):
                wp[i][j] = -math.inf
    y, w = [], []
    for i in range(n):
        e = [math.exp(x) for x in wp[i]]
        s = sum(e)
        wi = [x / s for x in e]
        w.append(wi)
        y.append([sum(wi[j] * v[j][c] for j in range(n)) for c in range(d)])
    return np.array(y), np.array(w), np.array(wp)


def _qkv(n, d, seed, scale=0.7):
    rng = np.random.default_rng(seed)
    return [rng.standard_normal((n, d)) * scale for _ in range(3)]


@pytest.mark.parametrize("n,d", [(1, 1), (2, 3), (5, 3), (7, 9), (12, 4)])
@pytest.mark.parametrize("scale", [1.0, 0.5])
def test_full_matches_brute_force(n, d, scale):
    q, k, v = _qkv(n, d, 10 * n + d)
    y, w, wp = brute_force(q.tolist(), k.tolist(), v.tolist(), scale)
    Y, _, W, S = oracle.attention_slice(q, k, v, oracle.FULL, scale, want_weights=True, want_scores=True)
    assert np.abs(S - wp).max() <= 1e-14
    assert np.abs(W - w).max() <= 1e-14
    assert np.abs(Y - y).max() <= 1e-13


@pytest.mark.parametrize("n,d", [(1, 2), (2, 3), (5, 3), (7, 9), (12, 4)])
def test_masked_matches_unmasked_then_masked_brute_force(n, d):
    q, k, v = _qkv(n, d, 100 + n)
    y, w, _ = brute_force(q.tolist(), k.tolist(), v.tolist(), 1.0, masked=True)
    Y, _, W, S = oracle.attention_slice(q, k, v, oracle.MASKED, 1.0, want_weights=True, want_scores=True)
    assert np.abs(Y - y).max() <= 1e-13
    assert np.abs(W - w).max() <= 1e-14
    iu = np.triu_indices(n, 1)
    assert np.all(W[iu] == 0.0)          # masked positions carry exactly zero weight
    assert np.all(np.isnan(S[iu]))       # and were never computed in phase 1
    assert not np.isnan(S[np.tril_indices(n)]).any()


@pytest.mark.parametrize("n,d", [(9, 5), (40, 16), (64, 64), (130, 7)])
def test_full_and_masked_match_library_softmax_and_matmul(n, d):
    # Special case that reduces to library routines; n != d and q != k catch a transposed operand.
    q, k, v = _qkv(n, d, n * d, scale=0.5)
    s = (q @ k.T) / math.sqrt(d)
    Y, _, _, _ = oracle.attention_slice(q, k, v, oracle.FULL, 1 / math.sqrt(d))
    assert np.abs(Y - scipy.special.softmax(s, axis=1) @ v).max() <= 1e-12
    s[np.triu_indices(n, 1)] = -np.inf
    Y, _, _, _ = oracle.attention_slice(q, k, v, oracle.MASKED, 1 / math.sqrt(d))
    assert np.abs(Y - scipy.special.softmax(s, axis=1) @ v).max() <= 1e-12


def test_weight_rows_sum_to_one():
    q, k, v = _qkv(50, 8, 3, scale=2.0)
    for scheme in (oracle.FULL, oracle.MASKED, oracle.SYMMETRIC):
        _, _, W, _ = oracle.attention_slice(q, k, v, scheme, 1.0, want_weights=True)
        assert np.abs(W.sum(axis=1) - 1.0).max() <= 1e-14
        assert (W >= 0).all()


def test_uniform_weights_closed_form():
    # q = 0 makes every score equal: FULL gives the mean of v, MASKED the running (prefix) mean.
    n, d = 23, 6
    _, k, v = _qkv(n, d, 5)
    q = np.zeros((n, d))
    Y, _, _, _ = oracle.attention_slice(q, k, v, oracle.FULL, 1.0)
    assert np.abs(Y - v.mean(axis=0)).max() <= 1e-14
    Y, _, _, _ = oracle.attention_slice(q, k, v, oracle.MASKED, 1.0)
    prefix = np.cumsum(v, axis=0) / np.arange(1, n + 1)[:, None]
    assert np.abs(Y - prefix).max() <= 1e-14


def test_masked_first_row_is_first_value_exactly():
    q, k, v = _qkv(17, 4, 8)
    Y, _, _, _ = oracle.attention_slice(q, k, v, oracle.MASKED, 1.0)
    assert np.array_equal(Y[0], v[0])


def test_one_dominant_key_selects_its_value():
    n, d = 11, 4
    q, k, v = _qkv(n, d, 9)
    q[:] = 0; k[:] = 0
    q[:, 0] = 1.0
    k[6, 0] = 800.0                      # score 800 against 0 elsewhere
    Y, _, _, _ = oracle.attention_slice(q, k, v, oracle.FULL, 1.0)
    assert np.abs(Y - v[6]).max() <= 1e-300 + 1e-15 * np.abs(v[6]).max()
    Y, _, _, _ = oracle.attention_slice(q, k, v, oracle.MASKED, 1.0)
    assert np.abs(Y[6:] - v[6]).max() <= 1e-15
    assert np.abs(Y[3] - v[:4].mean(axis=0)).max() <= 1e-15   # rows before key 6 never see it


def test_shift_invariance_of_softmax():
    # Adding the same vector t to every key shifts all scores of row i by q_i.t: weights unchanged.
    n, d = 19, 5
    q, k, v = _qkv(n, d, 12)
    t = np.random.default_rng(1).standard_normal(d)
    for scheme in (oracle.FULL, oracle.MASKED):
        Y0, _, _, _ = oracle.attention_slice(q, k, v, scheme, 1.0)
        Y1, _, _, _ = oracle.attention_slice(q, k + t, v, scheme, 1.0)
        assert np.abs(Y0 - Y1).max() <= 1e-12


def test_full_is_equivariant_under_key_value_permutation():
    n, d = 21, 4
    q, k, v = _qkv(n, d, 13)
    p = np.random.default_rng(2).permutation(n)
    Y0, _, _, _ = oracle.attention_slice(q, k, v, oracle.FULL, 1.0)
    Y1, _, _, _ = oracle.attention_slice(q, k[p].copy(), v[p].copy(), oracle.FULL, 1.0)
    assert np.abs(Y0 - Y1).max() <= 1e-13
    Y2, _, _, _ = oracle.attention_slice(q[p].copy(), k, v, oracle.FULL, 1.0)
    assert np.abs(Y0[p] - Y2).max() == 0.0


@pytest.mark.parametrize("n", [3, 4, 9, 10, 33])
@pytest.mark.parametrize("sel", [oracle.SEL_MINIMAL, oracle.SEL_PAPER])
def test_symmetric_scheme_equals_full_with_shared_vectors_bitwise(n, sel):
    d = 6
    x, _, _ = _qkv(n, d, 40 + n)
    Yf, _, Wf, Sf = oracle.attention_slice(x, x, x, oracle.FULL, 1.0, want_weights=True, want_scores=True)
    Ys, _, Ws, Ss = oracle.attention_slice(x, None if False else x, x, oracle.SYMMETRIC, 1.0, sel,
                                           want_weights=True, want_scores=True)
    assert np.array_equal(Sf, Sf.T)                     # Eq. 4: w'_ij = w'_ji
    assert np.array_equal(Ss, Sf) and np.array_equal(Ws, Wf) and np.array_equal(Ys, Yf)
    y, _, _ = brute_force(x.tolist(), x.tolist(), x.tolist(), 1.0)
    assert np.abs(Ys - y).max() <= 1e-13


def test_symmetric_paper_selection_is_cyclic_diagonals():
    # Sec. 4.2 items 2-4 for n = 5 (odd) and n = 4 (even): which w'_ij phase 1 computes.  Read off through
    # the census of a one-hot construction: with d = 1 the census counts selected positions.
    for n, want in ((5, 15), (4, 12), (6, 24), (7, 28)):
        x = np.ones((n, 1))
        _, c, _, _ = oracle.attention_slice(x, x, x, oracle.SYMMETRIC, 1.0, oracle.SEL_PAPER)
        assert c.mac1 == want


@pytest.mark.parametrize("scheme,sel", [(oracle.FULL, 0), (oracle.MASKED, 0), (oracle.SYMMETRIC, 0),
                                        (oracle.SYMMETRIC, 1)])
def test_row_subset_entry_matches_brute_force_and_slice(scheme, sel):
    B, n, H, d = 2, 13, 3, 5
    rng = np.random.default_rng(7)
    Q, K, V = (rng.standard_normal((B, n, H, d)) for _ in range(3))
    if scheme == oracle.SYMMETRIC:
        K = V = Q
    b, h = 1, 2
    rows = [0, 4, 12, 7]
    Y = oracle.attention_rows(Q, K, V, scheme, b, h, rows, scale=0.3, selection=sel)
    y, _, _ = brute_force(Q[b, :, h].tolist(), K[b, :, h].tolist(), V[b, :, h].tolist(), 0.3,
                          masked=(scheme == oracle.MASKED))
    assert np.abs(Y - y[rows]).max() <= 1e-13
    full, _ = oracle.attention_core(Q, K, V, scheme, 0.3, sel)
    assert np.array_equal(full[b, rows, h * d:(h + 1) * d], Y)


def test_projection_is_the_matrix_product():
    rng = np.random.default_rng(3)
    X = rng.standard_normal((2, 9, 7)); W = rng.standard_normal((7, 10))
    P = oracle.project(X, W)
    assert np.abs(P - np.matmul(X, W)).max() <= 1e-13
    ref = np.zeros((2, 9, 10))
    for b in range(2):
        for c in range(10):          # a differently ordered loop: column by column, k descending
            for r in range(9):
                acc = 0.0
                for kk in range(6, -1, -1):
                    acc += X[b, r, kk] * W[kk, c]
                ref[b, r, c] = acc
    assert np.abs(P - ref).max() <= 1e-13


def test_layer_splits_heads_by_column_blocks():
    # Sec. 3.1 multi-head remark: each head is its own set of projection matrices and runs the same phases.
    rng = np.random.default_rng(4)
    B, n, D, H, d = 2, 10, 6, 3, 4
    X = rng.standard_normal((B, n, D)) * 0.5
    Wq, Wk, Wv = (rng.standard_normal((D, H * d)) * 0.5 for _ in range(3))
    for scheme in (oracle.FULL, oracle.MASKED, oracle.SYMMETRIC):
        out, cnt = oracle.attention_layer(X, Wq, Wk, Wv, H, scheme)
        for b in range(B):
            for h in range(H):
                sl = slice(h * d, (h + 1) * d)
                q = X[b] @ Wq[:, sl]
                k = q if scheme == oracle.SYMMETRIC else X[b] @ Wk[:, sl]
                v = q if scheme == oracle.SYMMETRIC else X[b] @ Wv[:, sl]
                s = q @ k.T / math.sqrt(d)
                if scheme == oracle.MASKED:
                    s[np.triu_indices(n, 1)] = -np.inf
                want = scipy.special.softmax(s, axis=1) @ v
                assert np.abs(out[b, :, sl] - want).max() <= 1e-12
        per_head = d * n * (n + 1) // 2 if scheme != oracle.FULL else d * n * n
        assert cnt.mac1 == B * H * per_head


def test_block_is_sum_over_heads_of_head_output_times_its_rows_of_wo():
    # Output projection after the heads: z = sum_h y^(h) Wo[h*d:(h+1)*d, :], each y^(h) by library softmax/matmul.
    rng = np.random.default_rng(5)
    B, n, D, H, d = 2, 9, 6, 3, 4
    X = rng.standard_normal((B, n, D)) * 0.5
    Wq, Wk, Wv = (rng.standard_normal((D, H * d)) * 0.5 for _ in range(3))
    Wo = rng.standard_normal((H * d, D)) * 0.5
    for scheme in (oracle.FULL, oracle.MASKED, oracle.SYMMETRIC):
        z, y, _ = oracle.attention_block(X, Wq, Wk, Wv, Wo, H, scheme)
        assert z.shape == (B, n, D) and y.shape == (B, n, H * d)
        for b in range(B):
            want = np.zeros((n, D))
            for h in range(H):
                sl = slice(h * d, (h + 1) * d)
                q = X[b] @ Wq[:, sl]
                k = q if scheme == oracle.SYMMETRIC else X[b] @ Wk[:, sl]
                v = q if scheme == oracle.SYMMETRIC else X[b] @ Wv[:, sl]
                s = q @ k.T / math.sqrt(d)
                if scheme == oracle.MASKED:
                    s[np.triu_indices(n, 1)] = -np.inf
                want += (scipy.special.softmax(s, axis=1) @ v) @ Wo[sl, :]
            assert np.abs(z[b] - want).max() <= 1e-12


def test_block_special_output_matrices():
    rng = np.random.default_rng(6)
    B, n, D, H, d = 1, 7, 8, 2, 4
    X = rng.standard_normal((B, n, D)) * 0.5
    Wq, Wk, Wv = (rng.standard_normal((D, H * d)) * 0.5 for _ in range(3))
    y_ref, _ = oracle.attention_layer(X, Wq, Wk, Wv, H, oracle.MASKED)
    # identity: the block is the layer
    z, y, _ = oracle.attention_block(X, Wq, Wk, Wv, np.eye(H * d), H, oracle.MASKED)
    assert np.array_equal(y, y_ref) and np.abs(z - y_ref).max() <= 1e-15
    # a column selector picks one head's one component; zero gives zero
    E = np.zeros((H * d, D)); E[5, 2] = 1.0
    z, _, _ = oracle.attention_block(X, Wq, Wk, Wv, E, H, oracle.MASKED)
    want = np.zeros((B, n, D)); want[..., 2] = y_ref[..., 5]
    assert np.abs(z - want).max() <= 1e-15
    # linear in Wo; not transposed (a non-square Wo would not even fit the other way round)
    A = rng.standard_normal((H * d, 5)); Bm = rng.standard_normal((H * d, 5))
    za, _, _ = oracle.attention_block(X, Wq, Wk, Wv, A, H, oracle.FULL)
    zb, _, _ = oracle.attention_block(X, Wq, Wk, Wv, Bm, H, oracle.FULL)
    zc, _, _ = oracle.attention_block(X, Wq, Wk, Wv, 2.0 * A - 3.0 * Bm, H, oracle.FULL)
    assert za.shape == (B, n, 5) and np.abs(zc - (2.0 * za - 3.0 * zb)).max() <= 1e-12
    # masked: the first output vector sees only the first value vector, z_0 = sum_h v_0^(h) Wo_h
    zm, _, _ = oracle.attention_block(X, Wq, Wk, Wv, A, H, oracle.MASKED)
    assert np.abs(zm[0, 0] - (X[0, 0] @ Wv) @ A).max() <= 1e-13


def test_block_residual_is_added_elementwise():
    # z = residual + y Wo: with a zero output matrix the block returns the residual itself; with the residual moved to
    # the other side it is the block without one; a library sum-of-heads product plus X pins the usual case R = X
    rng = np.random.default_rng(8)
    B, n, D, H, d = 2, 6, 5, 2, 3
    X = rng.standard_normal((B, n, D)) * 0.5
    Wq, Wk, Wv = (rng.standard_normal((D, H * d)) * 0.5 for _ in range(3))
    Wo = rng.standard_normal((H * d, D)) * 0.5
    R = rng.standard_normal((B, n, D))
    z0, _, _ = oracle.attention_block(X, Wq, Wk, Wv, np.zeros((H * d, D)), H, oracle.MASKED, residual=R)
    assert np.array_equal(z0, R)
    z_plain, _, _ = oracle.attention_block(X, Wq, Wk, Wv, Wo, H, oracle.FULL)
    z_res, _, _ = oracle.attention_block(X, Wq, Wk, Wv, Wo, H, oracle.FULL, residual=R)
    assert np.abs((z_res - R) - z_plain).max() <= 1e-15
    z_x, _, _ = oracle.attention_block(X, Wq, Wk, Wv, Wo, H, oracle.FULL, residual=X)
    for b in range(B):
        want = X[b].copy()
        for h in range(H):
            sl = slice(h * d, (h + 1) * d)
            s_ = (X[b] @ Wq[:, sl]) @ (X[b] @ Wk[:, sl]).T / math.sqrt(d)
            want += (scipy.special.softmax(s_, axis=1) @ (X[b] @ Wv[:, sl])) @ Wo[sl, :]
        assert np.abs(z_x[b] - want).max() <= 1e-12


def test_bf16_rounding_agrees_with_generator_and_torch():
    import torch
    rng = np.random.default_rng(5)
    a = np.concatenate([rng.standard_normal(4096) * 3, [0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895314e38]])
    r = oracle.round_bf16(a)
    via_gen = inputs.bf16_bits_to_f64(inputs.to_bf16_bits(a))
    via_torch = torch.from_numpy(a.astype(np.float32)).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(r, via_gen)
    assert np.array_equal(r, via_torch)
    assert r[-3] == 1.0 and r[-2] == 1.015625          # ties go to the even neighbour
