"""GPU parity: moqae_route against the oracle (bit-exact maps away from near-ties)."""
import numpy as np
import pytest
import torch

from oracle import moqae_oracle as O
from paper_2506_07533_b200 import binding as mq
from paper_2506_07533_b200 import synth

pytestmark = pytest.mark.gpu

TAU = 1e-4      # a token whose top-2 logits differ by less than TAU * max|P| may flip in float32


def assert_map_matches(ref, got_map, got_votes, hid, W1, W2, W3, b0, chunk, dtype, abs_margin=None):
    """Exact map and votes on every chunk whose vote no near-tie token can change; on the others the
    votes may differ by at most the fragile tokens and the winner must be reachable by flipping
    them between their two best experts.  Returns the number of fragile chunks."""
    B, C = got_map.shape
    n_fragile_chunks = 0
    for b in range(B):
        for c in range(C):
            sl = slice(c * chunk, (c + 1) * chunk)
            thr = abs_margin if abs_margin is not None else TAU * np.maximum(ref["pmax"][b, sl], 1e-30)
            frag = np.where(ref["margin"][b, sl] < thr)[0]
            diff = got_votes[b, c].astype(np.int64) - ref["votes"][b, c]
            assert diff.sum() == 0
            assert np.abs(diff).sum() // 2 <= len(frag), (b, c, diff, len(frag))
            if len(frag) == 0:
                assert (diff == 0).all()
                assert got_map[b, c] == ref["map"][b, c]
            else:
                n_fragile_chunks += 1
                x = O.to_f64(synth.to_u16(hid)[b, sl][frag], dtype)
                P = O.router_logits(x, O.to_f64(synth.to_u16(W1), dtype),
                                    None if W2 is None else O.to_f64(synth.to_u16(W2), dtype),
                                    None if W3 is None else W3.numpy().astype(np.float64),
                                    b0.numpy().astype(np.float64))
                order = np.argsort(-P, axis=1, kind="stable")
                win = O.reachable_winners(ref["votes"][b, c], list(order[:, 0]), list(order[:, 1]))
                assert int(got_map[b, c]) in win
    return n_fragile_chunks


def check_route(B, T, D, chunk, dtype, gated, rf, seed, bias=None, w_std=0.02, weights=None, abs_margin=None):
    hid = synth.hidden_states(B, T, D, chunk, dtype, seed, "cpu")
    W1, W2, W3, b0 = weights or synth.router_weights(D, 4, dtype, seed + 1, "cpu", std=w_std, gated=gated)
    if bias is not None:
        b0 = torch.tensor(bias, dtype=torch.float32)
    ref = O.route(synth.to_u16(hid), dtype, chunk, synth.to_u16(W1),
                  None if W2 is None else synth.to_u16(W2), None if W3 is None else W3.numpy(),
                  b0.numpy(), rf_first_chunk=rf)
    C = T // chunk
    cfg = mq.make_config(n_layers=1, n_q_heads=8, n_kv_heads=8, chunk=chunk, dtype=dtype, d_in=D,
                         max_tokens=max(T, chunk), batch=B, rf_first_chunk=int(rf))
    cache = mq.moqae_cache_bind(cfg, [1, 1, 1, 1])
    votes_out = torch.full((B, max(C, 1), 4), -1, dtype=torch.int32, device="cuda")
    mq.moqae_route(cfg, hid.cuda(), T, W1.cuda(), None if W2 is None else W2.cuda(),
                   None if W3 is None else W3.cuda(), b0.cuda(), 0, cache, votes_out)
    torch.cuda.synchronize()
    got_map = cache.map[0, :, :C].cpu().numpy()
    got_votes = cache.votes[0, :, :C].cpu().numpy()
    if C:
        assert (votes_out[:, :C].cpu().numpy() == got_votes).all()
    n_fragile_chunks = assert_map_matches(ref, got_map, got_votes, hid, W1, W2, W3, b0, chunk, dtype, abs_margin)
    # slots and counts follow from the GPU's own map exactly
    slot, count = O.assign_slots(got_map)
    assert (cache.slot[0, :, :C].cpu().numpy() == slot).all()
    assert (cache.count[0].cpu().numpy() == count).all()
    if rf and C:
        assert (got_map[:, 0] == 3).all() and (got_votes[:, 0] == 0).all()
    return n_fragile_chunks, C * B, got_map


@pytest.mark.parametrize("gated", [False, True])
@pytest.mark.parametrize("dtype", [0, 1])
def test_route_config1_shape(gated, dtype):
    # config 1: hidden 1024, context 4096, chunk 128, weights ~ N(0, 0.02)
    nf, n, m = check_route(1, 4096, 1024, 128, dtype, gated, True, seed=100 + dtype)
    assert nf <= max(1, n // 4)


@pytest.mark.parametrize("chunk", [32, 64, 256, 512])
def test_route_chunk_sizes_and_tail(chunk):
    check_route(2, chunk * 5 + 7, 256, chunk, 1, True, True, seed=chunk, w_std=0.1)


def test_route_without_freezing_and_biased():
    _, _, m = check_route(2, 64 * 9, 128, 64, 0, False, False, seed=7, bias=[0.0, 0.0, 50.0, 0.0])
    assert (m == 2).all()                       # a dominant bias decides every chunk, chunk 0 included
    _, _, m = check_route(2, 64 * 9, 128, 64, 0, True, True, seed=8, bias=[50.0, 0.0, 0.0, 0.0])
    assert (m[:, 1:] == 0).all() and (m[:, 0] == 3).all()


def test_route_all_equal_logits_tie_goes_to_lowest_index():
    B, T, D, chunk = 1, 128, 64, 32
    hid = synth.hidden_states(B, T, D, chunk, 0, 5, "cpu")
    W1 = torch.zeros(D, 4, dtype=torch.float16)
    cfg = mq.make_config(n_layers=1, n_q_heads=8, n_kv_heads=8, chunk=chunk, dtype=0, d_in=D,
                         max_tokens=T, batch=B, rf_first_chunk=0)
    cache = mq.moqae_cache_bind(cfg, [1, 1, 1, 1])
    mq.moqae_route(cfg, hid.cuda(), T, W1.cuda(), None, None, None, 0, cache)
    torch.cuda.synchronize()
    assert (cache.map[0, 0, :4].cpu().numpy() == 0).all()
    assert (cache.votes[0, 0, :4].cpu().numpy() == np.array([32, 0, 0, 0])).all()


def test_route_short_and_empty_contexts():
    check_route(1, 20, 64, 32, 0, True, True, seed=1)       # no full chunk at all
    check_route(1, 32, 64, 32, 0, True, True, seed=2)       # exactly the frozen chunk


def test_routing_sharing_groups_are_independent_tables():
    B, T, D, chunk = 1, 32 * 6, 64, 32
    cfg = mq.make_config(n_layers=5, n_q_heads=8, n_kv_heads=8, chunk=chunk, dtype=1, d_in=D,
                         max_tokens=T, batch=B, rs_group=2)
    cache = mq.moqae_cache_bind(cfg, [1, 1, 1, 1])
    assert cache.n_groups == 3
    runs = []
    for g in range(3):
        hid = synth.hidden_states(B, T, D, chunk, 1, 50 + g, "cpu")
        W1, W2, W3, b0 = synth.router_weights(D, 4, 1, 60 + g, "cpu", std=0.2)
        mq.moqae_route(cfg, hid.cuda(), T, W1.cuda(), W2.cuda(), W3.cuda(), b0.cuda(), g, cache)
        ref = O.route(synth.to_u16(hid), 1, chunk, synth.to_u16(W1), synth.to_u16(W2), W3.numpy(), b0.numpy())
        runs.append((ref, hid, W1, W2, W3, b0))
    torch.cuda.synchronize()
    for g, (ref, hid, W1, W2, W3, b0) in enumerate(runs):
        # every group's table holds its own router's result: exact away from near-ties
        got = cache.map[g, :, :6].cpu().numpy()
        assert_map_matches(ref, got, cache.votes[g, :, :6].cpu().numpy(), hid, W1, W2, W3, b0, chunk, 1)
        assert (got[:, 0] == 3).all()
    assert any((runs[0][0]["map"] != runs[g][0]["map"]).any() for g in (1, 2))   # the tables do differ


@pytest.mark.parametrize("D", [32, 96, 160, 2080])
def test_route_input_widths_that_are_not_whole_boxes(D):
    # the hidden rows arrive in 64-channel boxes: widths below one box and with a ragged last box
    check_route(2, 64 * 4 + 3, D, 64, 1, True, True, seed=D, w_std=0.1)


def test_three_expert_set_through_a_masked_logit():
    # the {2, 4, 16}-bit expert set of the ablation: zero weights and an unreachable bias for the
    # 8-bit expert; the GPU router must never choose it and must match the oracle elsewhere
    D, chunk, dtype = 256, 64, 1
    W1, W2, W3, b = synth.router_weights(D, 3, dtype, 91, "cpu", std=0.1)
    keep = [0, 1, 3]
    W1_4 = torch.zeros(D, 4, dtype=W1.dtype); W1_4[:, keep] = W1
    W2_4 = torch.zeros(D, 4, dtype=W2.dtype); W2_4[:, keep] = W2
    W3_4 = torch.zeros(4, 4)
    for i, ki in enumerate(keep):
        for j, kj in enumerate(keep):
            W3_4[ki, kj] = W3[i, j]
    b_4 = torch.full((4,), -3.0e38); b_4[keep] = b
    # the masked logit would blow up a tolerance relative to max|P|: near-ties are judged against
    # the size of the live logits (a few units) instead
    n_frag, n_chunks, m = check_route(2, chunk * 12 + 9, D, chunk, dtype, True, True, seed=90,
                                      weights=(W1_4, W2_4, W3_4, b_4), abs_margin=1e-3)
    assert not (m == 2).any() and len(np.unique(m)) > 1 and n_frag < n_chunks // 2


def test_table_validator_reports_a_corrupted_slot_table():
    # tables written by the router pass the validator; one overwritten slot entry is found
    B, T, D, chunk = 2, 64 * 9 + 5, 64, 64
    cfg = mq.make_config(n_layers=1, n_q_heads=2, n_kv_heads=2, chunk=chunk, dtype=1, d_in=D, max_tokens=T, batch=B)
    cache = mq.moqae_cache_bind(cfg, [9, 9, 9, 9])
    hid = synth.hidden_states(B, T, D, chunk, 1, 77, "cuda")
    W1, W2, W3, b0 = synth.router_weights(D, 4, 1, 78, "cuda", std=0.2)
    mq.moqae_route(cfg, hid, T, W1, W2, W3, b0, 0, cache)
    assert mq.moqae_validate_tables(cfg, cache, T)[0] == mq.OK
    cache.slot[0, 1, 4] += 3
    assert mq.moqae_validate_tables(cfg, cache, T) == (mq.ERR_CORRUPT_TABLE, 1, 4)
    assert mq.moqae_validate_tables(cfg, cache, 4 * chunk)[0] == mq.ERR_CORRUPT_TABLE      # the counts describe 9 chunks
