"""Pins for the oracle's router (Eq. 1, Eq. 2, routing freezing / sharing)."""
import itertools
import os

import numpy as np
import pytest

from oracle import moqae_oracle as O

RS = np.random.RandomState


def f16bits(a):
    return np.asarray(a, dtype=np.float16).view(np.uint16)


def test_router_parameter_size_matches_paper():
    path = os.path.join(os.path.dirname(__file__), "golden", "router_param_bytes.txt")
    row = [l for l in open(path) if not l.startswith("#")][0].split()
    D, M, bpp, kb, tol = int(row[0]), int(row[1]), int(row[2]), float(row[3]), float(row[4])
    n_params = 2 * D * M + M * M           # W1, W2: D x M ; W3: M x M
    assert abs(n_params * bpp / 1000.0 - kb) <= tol
    # the literal "W3 in R^{D x M}" would give 3*D*M params = 2.3 KB: rejected by the same figure
    assert abs(3 * D * M * bpp / 1000.0 - kb) > tol


def test_eq1_gated_form_by_hand():
    # one token, D = 2, M = 2, numbers small enough to evaluate by hand
    x = np.array([[1.0, 2.0]])
    W1 = np.array([[1.0, 0.0], [0.0, 1.0]])          # u = (1, 2)
    W2 = np.array([[2.0, 1.0], [0.0, -1.0]])         # v = (2, 1-2) = (2, -1)
    W3 = np.array([[1.0, 0.0], [0.0, 3.0]])
    P = O.router_logits(x, W1, W2, W3)
    a = np.array([1.0 * 2.0, 2.0 * -1.0])            # product first ...
    silu = a / (1.0 + np.exp(-a))                    # ... activation after
    assert np.allclose(P, [[silu[0], 3.0 * silu[1]]], rtol=0, atol=1e-15)
    # SwiGLU ordering (activation on one factor only) would differ: guards the reading
    swiglu = (np.array([1.0, 2.0]) / (1 + np.exp(-np.array([1.0, 2.0])))) * np.array([2.0, -1.0])
    assert not np.allclose(P, [[swiglu[0], 3 * swiglu[1]]])


def test_linear_mode_equals_library_gemv():
    rs = RS(0)
    x = rs.randn(50, 64)
    W = rs.randn(64, 4)
    b = rs.randn(4).astype(np.float32)
    P = O.router_logits(x, W, None, None, b)
    ref = np.einsum("nd,dm->nm", x, W) + b.astype(np.float64)
    assert np.allclose(P, ref, atol=1e-12)
    assert (O.token_experts(P) == ref.argmax(1)).all()


@pytest.mark.parametrize("N,M", [(1, 2), (2, 3), (3, 3), (4, 4), (4, 2)])
def test_vote_brute_force(N, M):
    # every assignment of N tokens to M experts against a literal restatement of Eq. 2
    for e in itertools.product(range(M), repeat=N):
        votes, r = O.chunk_vote(np.array(e), M)
        counts = [sum(1 for i in range(N) if e[i] == k) for k in range(M)]
        best = max(counts)
        expect = min(k for k in range(M) if counts[k] == best)   # ties -> lowest index
        assert list(votes) == counts and r == expect


def test_token_argmax_ties_pick_lowest_index():
    P = np.array([[1.0, 1.0, 0.0, 1.0], [0.0, 2.0, 2.0, 1.0], [3.0, 3.0, 3.0, 3.0], [0, 0, 0, 1.0]])
    assert list(O.token_experts(P)) == [0, 1, 0, 3]


def _route_small(rf, T=100, N=32, B=2, D=16, seed=1, gated=True):
    rs = RS(seed)
    hid = f16bits(rs.randn(B, T, D))
    W1 = f16bits(rs.randn(D, 4) * 0.5)
    W2 = f16bits(rs.randn(D, 4) * 0.5) if gated else None
    W3 = rs.randn(4, 4).astype(np.float32) if gated else None
    bias = rs.randn(4).astype(np.float32) * 0.1
    return hid, W1, W2, W3, bias, O.route(hid, 0, N, W1, W2, W3, bias, rf_first_chunk=rf)


def test_route_chunking_tail_and_freezing():
    hid, W1, W2, W3, bias, r = _route_small(True)
    assert r["map"].shape == (2, 3)                     # 100 // 32 chunks; 4 tail tokens unrouted
    assert (r["map"][:, 0] == 3).all()                  # frozen first chunk -> 16-bit expert
    assert (r["votes"][:, 0] == 0).all()
    assert (r["votes"][:, 1:].sum(-1) == 32).all()      # every routed token votes once
    # freezing does not depend on the weights
    r2 = O.route(hid, 0, 32, f16bits(np.zeros((16, 4))), None, None,
                 np.array([5, 0, 0, 0], np.float32), rf_first_chunk=True)
    assert (r2["map"][:, 0] == 3).all() and (r2["map"][:, 1:] == 0).all()
    # without freezing the first chunk is routed like the others
    r3 = O.route(hid, 0, 32, f16bits(np.zeros((16, 4))), None, None,
                 np.array([5, 0, 0, 0], np.float32), rf_first_chunk=False)
    assert (r3["map"] == 0).all()


def test_route_matches_per_chunk_recomputation():
    hid, W1, W2, W3, bias, r = _route_small(False, seed=3)
    x = hid.view(np.float16).astype(np.float64)
    for b in range(2):
        for c in range(3):
            xs = x[b, c * 32:(c + 1) * 32]
            a = (xs @ W1.view(np.float16).astype(np.float64)) * (xs @ W2.view(np.float16).astype(np.float64))
            P = (a / (1 + np.exp(-a))) @ W3.astype(np.float64) + bias.astype(np.float64)
            cnt = np.bincount(P.argmax(1), minlength=4)
            assert (cnt == r["votes"][b, c]).all()
            assert r["map"][b, c] == cnt.argmax()


def test_routing_sharing_groups():
    # groups of gs consecutive blocks share the first block's map; last group may be short
    assert [O.layer_group(l, 3) for l in range(8)] == [0, 0, 0, 1, 1, 1, 2, 2]
    assert O.n_groups(32, 3) == 11 and O.n_groups(40, 4) == 10 and O.n_groups(5, 1) == 5


def test_slots_dense_and_increasing():
    rs = RS(5)
    m = rs.randint(0, 4, size=(3, 40)).astype(np.uint8)
    slot, count = O.assign_slots(m)
    for b in range(3):
        for w in range(4):
            s = slot[b][m[b] == w]
            assert list(s) == list(range(len(s))) and count[b, w] == len(s)


def test_reachable_winners():
    v = np.array([5, 5, 0, 0])
    assert O.reachable_winners(v, [], []) == {0}
    assert O.reachable_winners(v, [0], [1]) == {0, 1}
    assert O.reachable_winners(np.array([9, 1, 0, 0]), [0], [1]) == {0}


@pytest.mark.parametrize("nf", [1, 5, 12, 13, 16])
def test_reachable_winners_against_enumeration_of_every_flip_pattern(nf):
    # brute force written out here: try all 2^nf subsets of flipped tokens (also beyond a dozen
    # tokens, where an earlier version of the function fell back to a superset)
    rs = RS(40 + nf)
    for trial in range(6):
        votes = rs.randint(0, 6, size=4) + np.array([nf, 0, 0, 0]) // 2
        cur = [int(x) for x in rs.randint(0, 4, size=nf)]
        alt = [int((c + rs.randint(1, 4)) % 4) for c in cur]
        for c in cur:
            votes[c] += 1                       # every fragile token's current vote is in the histogram
        want = set()
        for mask in range(1 << nf):
            v = votes.astype(np.int64).copy()
            for i in range(nf):
                if mask >> i & 1:
                    v[cur[i]] -= 1
                    v[alt[i]] += 1
            want.add(int(np.argmax(v)))
        assert O.reachable_winners(votes, cur, alt) == want


def _embed_three_experts(W1, W2, W3, bias):
    """A {2, 4, 16}-bit router written as the four-expert one: the 8-bit expert gets zero weights
    and a logit no token can choose."""
    keep = [0, 1, 3]
    W1_4 = np.zeros((W1.shape[0], 4), W1.dtype); W1_4[:, keep] = W1
    W2_4 = np.zeros((W2.shape[0], 4), W2.dtype); W2_4[:, keep] = W2
    W3_4 = np.zeros((4, 4), np.float32); W3_4[np.ix_(keep, keep)] = W3
    b_4 = np.full(4, -3.0e38, np.float32); b_4[keep] = bias
    return W1_4, W2_4, W3_4, b_4


def test_three_expert_set_is_the_four_expert_router_with_one_logit_masked():
    # the ablation with M = 3 experts {2, 4, 16 bits} (Section 4.4): its router, run with M = 3 in
    # the oracle, chooses exactly what the M = 4 router chooses when the 8-bit expert is masked
    rs = RS(11)
    B, T, D, N = 2, 32 * 9 + 5, 24, 32
    hid = f16bits(rs.randn(B, T, D))
    W1, W2 = f16bits(rs.randn(D, 3) * 0.5), f16bits(rs.randn(D, 3) * 0.5)
    W3, bias = rs.randn(3, 3).astype(np.float32), (rs.randn(3) * 0.1).astype(np.float32)
    r3 = O.route(hid, 0, N, W1, W2, W3, bias, rf_first_chunk=True)
    r4 = O.route(hid, 0, N, *_embed_three_experts(W1, W2, W3, bias), rf_first_chunk=True)
    widths = np.array([0, 1, 3], np.uint8)              # expert index of the 3-set -> index of the 4-set
    assert (widths[r3["map"]] == r4["map"]).all()
    assert (r4["votes"][:, :, [0, 1, 3]] == r3["votes"]).all() and (r4["votes"][:, :, 2] == 0).all()
    assert (r4["map"][:, 0] == 3).all() and len(np.unique(r4["map"])) > 1
