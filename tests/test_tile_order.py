"""The carry chain's forward-progress argument, checked on the host: the scan kernels launch a
(G, B, K) grid (x = 64-channel group, y = batch row, z = tile along time) and a tile only ever waits
for tiles of its own (group, batch row) with a smaller k.  With x fastest and z slowest, every such
predecessor has a smaller linear block index, so it was handed to an SM no later than its waiter.
The window each tile reads (the last checkpoint's carry-in and the aggregates since) is also
enumerated here and must only name earlier tiles."""
import itertools

import pytest

K_WINDOW = 7          # every 7th tile of a chain is a checkpoint (kWindow in the kernel)


def linear_index(g, b, k, G, B):
    return (k * B + b) * G + g


def window(k):
    """(checkpoint tile whose carry-in is read or None for the call's initial state, aggregates read)."""
    cpt = K_WINDOW * ((k - 1) // K_WINDOW) if k > 0 else 0
    return (cpt if cpt > 0 else None), list(range(cpt, k))


@pytest.mark.parametrize("G,B,K", [(1, 1, 1), (12, 8, 16), (12, 1, 32), (3, 5, 23), (12, 16, 64)])
def test_predecessors_have_smaller_linear_indices(G, B, K):
    for g, b, k in itertools.product(range(G), range(B), range(K)):
        me = linear_index(g, b, k, G, B)
        cpt, aggs = window(k)
        for kk in aggs + ([cpt] if cpt is not None else []):
            assert 0 <= kk < k
            assert linear_index(g, b, kk, G, B) < me


def test_window_is_a_function_of_k_alone_and_bounded():
    for k in range(0, 200):
        cpt, aggs = window(k)
        assert len(aggs) <= K_WINDOW                       # at most seven aggregates are folded
        if k > 0:
            assert aggs[-1] == k - 1 and aggs == list(range(aggs[0], k))
        assert (cpt is None) == (k <= K_WINDOW)            # the first seven tiles start from the initial state
        if cpt is not None:
            assert cpt % K_WINDOW == 0 and aggs[0] == cpt   # the window starts at the checkpoint


def test_checkpoint_chain_is_the_only_serial_dependency():
    """A checkpoint's carry-in depends on the previous checkpoint's; everything else a tile reads
    (aggregates) is published before its writer waits for anything."""
    K = 100
    depth = {}
    for k in range(K):
        cpt, _ = window(k)
        depth[k] = 0 if cpt is None else depth[cpt] + 1
    assert depth[K - 1] == (K - 2) // K_WINDOW
    assert max(depth.values()) == (K - 2) // K_WINDOW
