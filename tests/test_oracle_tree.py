"""Pins for the oracle's token tree of the beams and its greedy verification.

The tree is checked against a hand-built case, against the set of distinct beam prefixes and
by walking parents back; the tree walk against the single-path verification of every beam (the
tree must do as well as the best beam and take its token) and against the one-beam case.
"""
import pytest
import torch

import oracle


def test_hand_built_tree():
    beams = torch.tensor([[[5, 6, 7], [5, 6, 8], [5, 9, 7], [4, 6, 7]]], dtype=torch.int32)
    t = oracle.beam_tree(beams, torch.tensor([3], dtype=torch.int32))
    assert t.n_nodes.tolist() == [9]
    assert t.node_token[0, :9].tolist() == [5, 6, 7, 8, 9, 7, 4, 6, 7]
    assert t.node_parent[0, :9].tolist() == [-1, 0, 1, 1, 0, 4, -1, 6, 7]
    assert t.node_depth[0, :9].tolist() == [0, 1, 2, 2, 1, 2, 0, 1, 2]
    assert t.beam_node[0].tolist() == [[0, 1, 2], [0, 1, 3], [0, 4, 5], [6, 7, 8]]
    assert (t.node_token[0, 9:] == -1).all() and (t.node_parent[0, 9:] == -1).all()


def _random_beams(B, W, L, V, seed, live=None):
    g = torch.Generator().manual_seed(seed)
    beams = torch.randint(0, V, (B, W, L), generator=g, dtype=torch.int32)
    # make prefixes collide: later beams copy a random-length prefix of an earlier one
    for b in range(B):
        for w in range(1, W):
            src = int(torch.randint(0, w, (1,), generator=g))
            k = int(torch.randint(0, L + 1, (1,), generator=g))
            beams[b, w, :k] = beams[b, src, :k]
    path_len = torch.randint(1, L + 1, (B,), generator=g, dtype=torch.int32)
    for b in range(B):
        beams[b, :, int(path_len[b]):] = -1
        if live is not None:
            beams[b, live:, :] = -1
    return beams, path_len


@pytest.mark.parametrize("W,L,V,live", [(1, 6, 50, None), (4, 5, 3, None), (8, 7, 4, 5), (16, 4, 2, None)])
def test_tree_nodes_are_the_distinct_prefixes_and_parents_walk_back_to_the_beams(W, L, V, live):
    B = 5
    beams, path_len = _random_beams(B, W, L, V, seed=W * 10 + L, live=live)
    t = oracle.beam_tree(beams, path_len)
    for b in range(B):
        m = int(path_len[b])
        prefixes = set()
        for w in range(W):
            if beams[b, w, 0] < 0:
                continue
            for i in range(1, m + 1):
                prefixes.add(tuple(beams[b, w, :i].tolist()))
        n = int(t.n_nodes[b])
        assert n == len(prefixes)
        assert t.beam_node[b, 0, :m].tolist() == list(range(m))          # the rank-0 path comes first
        for w in range(W):
            for i in range(L):
                node = int(t.beam_node[b, w, i])
                if beams[b, w, 0] < 0 or i >= m:
                    assert node == -1
                    continue
                toks, x = [], node
                while x >= 0:
                    toks.append(int(t.node_token[b, x]))
                    assert t.node_depth[b, x] == i - (len(toks) - 1)
                    x = int(t.node_parent[b, x])
                assert toks[::-1] == beams[b, w, :i + 1].tolist()
        assert (t.node_parent[b, :n] < torch.arange(n)).all()              # parents come before children


def _consistent_target(tree, B, N, V, seed):
    """Target rows that depend only on the context (the tokens up to a node): what a causal model gives."""
    x = torch.empty((B, 1 + N, V))
    for b in range(B):
        for ctx in range(-1, int(tree.n_nodes[b])):
            toks, n = [], ctx
            while n >= 0:
                toks.append(int(tree.node_token[b, n]))
                n = int(tree.node_parent[b, n])
            g = torch.Generator().manual_seed(hash((seed, b, tuple(toks[::-1]))) % (2 ** 31))
            x[b, 1 + ctx] = torch.randn(V, generator=g)
        x[b, 1 + int(tree.n_nodes[b]):] = float("nan")                     # slots without a node are never read
    return x


@pytest.mark.parametrize("W,L,V", [(1, 6, 5), (4, 5, 3), (8, 6, 2), (6, 4, 4)])
def test_tree_walk_equals_the_best_single_path_verification(W, L, V):
    B = 6
    beams, path_len = _random_beams(B, W, L, V, seed=W + L)
    tree = oracle.beam_tree(beams, path_len)
    N = W * L
    x = _consistent_target(tree, B, N, V, seed=7)
    out = oracle.verify_tree(x, tree, L)
    assert (out.row_status == 0).all()
    for b in range(B):
        m = int(path_len[b])
        best = (-1, None)
        for w in range(W):
            # the rows this beam alone would be verified against: after the prefix, after its 1st token, ...
            rows = [0] + [1 + int(tree.beam_node[b, w, i]) for i in range(m)]
            tgt = x[b, rows].unsqueeze(0)                                  # [1, m + 1, V]: a bonus row exists
            single = oracle.verify(tgt, None, beams[b:b + 1, w, :m], torch.tensor([m], dtype=torch.int32))
            if int(single.accepted_len) > best[0]:
                best = (int(single.accepted_len), int(single.next_token))
        assert int(out.accepted_len[b]) == best[0] and int(out.next_token[b]) == best[1]
        acc = int(out.accepted_len[b])
        nodes = out.accepted_node[b, :acc].tolist()
        assert (out.accepted_node[b, acc:] == -1).all()
        for i, n in enumerate(nodes):                                      # a root-to-node path, depth by depth
            assert int(tree.node_depth[b, n]) == i
            assert int(tree.node_parent[b, n]) == (nodes[i - 1] if i else -1)
            assert int(tree.node_token[b, n]) == int(x[b, 1 + (nodes[i - 1] if i else -1)].argmax())


def test_nonfinite_rows_flag_existing_nodes_only():
    """Written by hand: two beams (5,6) and (5,7) give nodes 0:5, 1:6 (child of 0), 2:7 (child of 0);
    rows 0..3 exist, rows 4.. are unused slots."""
    beams = torch.tensor([[[5, 6], [5, 7]]], dtype=torch.int32)
    tree = oracle.beam_tree(beams, torch.tensor([2], dtype=torch.int32))
    assert tree.n_nodes.tolist() == [3]
    V, N = 8, 4
    x = torch.zeros((1, 1 + N, V))
    x[0, 0, 5] = 1.0          # after the prefix: token 5 -> node 0
    x[0, 1, 6] = 1.0          # after node 0: token 6 -> node 1
    x[0, 2, 3] = 1.0          # after node 1 (a leaf): bonus token 3
    x[0, 3, 2] = 1.0          # after node 2: never walked
    x[0, 4, :] = float("nan")  # unused slot
    o = oracle.verify_tree(x, tree, 2)
    assert o.accepted_len.tolist() == [2] and o.accepted_node[0].tolist() == [0, 1] and o.next_token.tolist() == [3]
    assert o.row_status.tolist() == [0]                       # the NaN slot has no node: not read, not flagged
    for val in (float("nan"), float("inf")):
        y = x.clone()
        y[0, 3, 0] = val                                      # the row of node 2 exists but the walk never reads it
        o = oracle.verify_tree(y, tree, 2)
        assert o.row_status.tolist() == [oracle.NONFINITE_INPUT]
        assert o.accepted_len.tolist() == [2] and o.next_token.tolist() == [3]      # the walk itself is unchanged
    y = x.clone()
    y[0, 3, 0] = -float("inf")                                # masking is legal
    assert oracle.verify_tree(y, tree, 2).row_status.tolist() == [0]
