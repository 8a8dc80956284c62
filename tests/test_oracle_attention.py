"""Pins of the oracle's Eq. 3 (attention over the routed tokens) against what the mathematics
fixes: the dense special case computed by a library softmax, a single-token route, invariance
under slot order, duplicates and logit shifts, and a hand-worked two-token case."""
import numpy as np
import torch

from oracle import routerelay_oracle as O


def _rand(seed, n_q=5, tokens=24, dh=8):
    rng = np.random.default_rng(seed)
    return rng.standard_normal((n_q, dh)), rng.standard_normal((tokens, dh)), rng.standard_normal((tokens, dh))


def test_all_chunks_selected_is_dense_softmax_attention():
    q, k, v = _rand(1)
    T = 4
    routes = np.tile(np.arange(6, dtype=np.int32), (5, 1))
    got = O.routed_attention(q, k, v, routes, T, 0.3)
    want = torch.softmax(torch.from_numpy(q) @ torch.from_numpy(k).T * 0.3, dim=-1) @ torch.from_numpy(v)
    np.testing.assert_allclose(got, want.numpy(), rtol=1e-12, atol=1e-12)


def test_single_token_route_returns_that_value_row():
    q, k, v = _rand(2)
    routes = np.full((5, 3), -1, np.int32)
    routes[:, 1] = [0, 5, 23, 7, 11]
    got = O.routed_attention(q, k, v, routes, 1, 1.7)
    np.testing.assert_allclose(got, v[[0, 5, 23, 7, 11]], rtol=0, atol=1e-15)


def test_slot_order_duplicates_and_empty_rows():
    q, k, v = _rand(3)
    a = np.array([[4, 1, -1, 2]] * 5, np.int32)
    b = np.array([[2, -1, 4, 1]] * 5, np.int32)
    np.testing.assert_array_equal(O.routed_attention(q, k, v, a, 4, 0.5),
                                  O.routed_attention(q, k, v, b, 4, 0.5))
    empty = np.full((5, 2), -1, np.int32)
    assert not O.routed_attention(q, k, v, empty, 4, 0.5).any()


def test_hand_worked_two_tokens_and_sequence_clipping():
    # one query, two selected tokens with logits ln 1 and ln 3: weights 1/4 and 3/4
    q = np.array([[1.0, 0.0]])
    k = np.array([[0.0, 5.0], [np.log(3.0), -2.0], [9.0, 9.0]])
    v = np.array([[4.0, 0.0], [0.0, 8.0], [100.0, 100.0]])
    got = O.routed_attention(q, k, v, np.array([[0]], np.int32), 2, 1.0)
    np.testing.assert_allclose(got, [[1.0, 6.0]], rtol=1e-14)
    # chunk 1 of size 2 covers tokens 2, 3: token 3 does not exist and is clipped
    got = O.routed_attention(q, k, v, np.array([[1]], np.int32), 2, 1.0)
    np.testing.assert_allclose(got, [[100.0, 100.0]], rtol=1e-14)


def test_adding_a_common_vector_to_all_keys_changes_nothing():
    q, k, v = _rand(4)
    routes = np.array([[0, 3, 5]] * 5, np.int32)
    base = O.routed_attention(q, k, v, routes, 4, 0.8)
    shifted = O.routed_attention(q, k + 3.0, v, routes, 4, 0.8)   # logits of a row shift together
    np.testing.assert_allclose(base, shifted, rtol=1e-9, atol=1e-12)
