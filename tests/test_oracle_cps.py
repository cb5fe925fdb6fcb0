"""Pins for the oracle's causal-consistency path search (Eq. 8, beam search, EOS early stop).

The beam is checked against exhaustive enumeration of every lattice path,
against an exact dynamic-programming (Viterbi) optimum, against special cases
that reduce to per-position argmax or a greedy walk, and against Eq. 8
re-evaluated directly on the returned paths.
"""
import itertools
import math

import numpy as np
import pytest
import torch

import oracle


def _lattice(L, V, K, seed, tau=0.0, eos_id=-1, B=1):
    g = torch.Generator().manual_seed(seed)
    x = 2.0 * torch.randn((B, L, V), generator=g)
    lat = oracle.lattice_build(x, K, tau=tau, eos_id=eos_id)
    table = -8.0 * torch.rand((V, V), generator=g)
    prev = torch.randint(0, V, (B,), generator=g, dtype=torch.int32)
    return x, lat, table, prev


def _eq8(lat, table, prev, b, ids, slots, lam):
    """Eq. 8 of one path in double, straight from the definition."""
    s, p = 0.0, int(prev[b])
    for i, (t, k) in enumerate(zip(ids, slots)):
        ldlm = float(lat.cand_logit[b, i, k]) - float(lat.lse64[b, i])
        s += lam * ldlm + (1.0 - lam) * float(table[p, t])
        p = t
    return s


def _search(lat, table, prev, W, lam, eos_id=-1):
    V = table.shape[0]
    return oracle.cps_search(lat.cand_id, lat.cand_logit, lat.lse64, lat.cand_count, prev, table,
                             W=W, lam=lam, eos_id=eos_id, proxy_kind=1, V=V)


@pytest.mark.parametrize("L,K,seed,tau", [(3, 4, 0, 0.0), (4, 3, 1, 0.0), (5, 2, 2, 0.0),
                                          (6, 2, 3, 0.0), (4, 4, 4, 0.6), (5, 3, 5, 0.7)])
def test_wide_beam_equals_brute_force_over_all_paths(L, K, seed, tau):
    V, lam = 12, 0.5
    _, lat, table, prev = _lattice(L, V, K, seed, tau=tau)
    W = K ** (L - 1)                                      # nothing is ever cut before the last depth
    out = _search(lat, table, prev, W, lam)
    counts = lat.cand_count[0].tolist()
    scored = []
    for slots in itertools.product(*[range(c) for c in counts]):
        ids = [int(lat.cand_id[0, i, k]) for i, k in enumerate(slots)]
        scored.append((_eq8(lat, table, prev, 0, ids, slots, lam), ids))
    scored.sort(key=lambda t: -t[0])
    assert len(scored) == math.prod(counts)
    assert abs(out.path_score.item() - scored[0][0]) < 1e-4
    if scored[0][0] - scored[1][0] > 1e-4:                # unique maximum: same path
        assert out.path[0].tolist() == scored[0][1]
    # the kept beams are the top-W of ALL paths (scores only; order within 1e-4)
    nb = min(W, len(scored))
    got = out.beam_score[0, :nb].double().numpy()
    want = np.array([s for s, _ in scored[:nb]])
    assert np.allclose(got, want, atol=1e-4)


def _viterbi(lat, table, prev, lam):
    """Exact optimum of Eq. 8 over the bigram lattice by dynamic programming (batch row 0)."""
    L = lat.cand_id.shape[1]
    best = None
    for i in range(L):
        c = int(lat.cand_count[0, i])
        cur = []
        for k in range(c):
            t = int(lat.cand_id[0, i, k])
            ldlm = float(lat.cand_logit[0, i, k]) - float(lat.lse64[0, i])
            if i == 0:
                cur.append(lam * ldlm + (1 - lam) * float(table[int(prev[0]), t]))
            else:
                cur.append(max(best[j] + lam * ldlm +
                               (1 - lam) * float(table[int(lat.cand_id[0, i - 1, j]), t])
                               for j in range(len(best))))
        best = cur
    return max(best)


@pytest.mark.parametrize("seed", range(4))
def test_viterbi_bound_and_equality(seed):
    L, K, V, lam = 6, 3, 20, 0.4
    _, lat, table, prev = _lattice(L, V, K, 10 + seed)
    opt = _viterbi(lat, table, prev, lam)
    last = -float("inf")
    for W in (1, 2, 4, 16, K ** (L - 1)):
        s = _search(lat, table, prev, W, lam).path_score.item()
        assert s <= opt + 1e-4                            # no beam beats the exact optimum
        last = s
    assert abs(last - opt) < 1e-4                         # the full-width beam reaches it


def test_lambda_one_returns_per_position_top1():
    L, K, V = 7, 4, 30
    for W in (1, 3, 8):
        _, lat, table, prev = _lattice(L, V, K, 20 + W, B=2)
        out = _search(lat, table, prev, W, 1.0)
        assert torch.equal(out.path, lat.cand_id[:, :, 0])
        assert (out.path_slot == 0).all() and (out.path_len == L).all()


def test_width_one_is_a_greedy_walk():
    L, K, V, lam = 6, 4, 25, 0.3
    _, lat, table, prev = _lattice(L, V, K, 30)
    out = _search(lat, table, prev, 1, lam)
    p, walk = int(prev[0]), []
    for i in range(L):
        steps = []
        for k in range(int(lat.cand_count[0, i])):
            t = int(lat.cand_id[0, i, k])
            g = float(lat.cand_logit[0, i, k]) - float(lat.cand_logit[0, i, 0])
            steps.append((lam * g + (1 - lam) * float(table[p, t]), -t, t))
        p = max(steps)[2]
        walk.append(p)
    assert out.path[0].tolist() == walk


@pytest.mark.parametrize("W", [1, 2, 5, 16])
def test_invariants_scores_sorted_eq8_recomputed_prefix_consistency(W):
    L, K, V, lam = 8, 4, 40, 0.5
    _, lat, table, prev = _lattice(L, V, K, 40 + W, B=3)
    out = _search(lat, table, prev, W, lam)
    cum = out.beam_cum
    assert (cum[:, :-1] >= cum[:, 1:]).all() if W > 1 else True       # ranking quantity sorted
    bs = out.beam_score.double()
    assert (bs[:, :-1] >= bs[:, 1:] - 1e-5).all() if W > 1 else True  # Eq. 8 values non-increasing
    for b in range(3):
        assert out.path_len[b].item() == L
        assert out.path[b].tolist() == out.beam_ids[b, 0].tolist()
        for w in range(min(W, K)):
            ids = out.beam_ids[b, w].tolist()
            slots = []
            for i, t in enumerate(ids):                   # every token is a candidate of its position
                row = lat.cand_id[b, i, :int(lat.cand_count[b, i])].tolist()
                assert t in row
                slots.append(row.index(t))
            assert abs(_eq8(lat, table, prev, b, ids, slots, lam) - out.beam_score[b, w].item()) < 1e-4
        assert [int(lat.cand_id[b, i, s]) for i, s in enumerate(out.path_slot[b].tolist())] == \
            out.path[b].tolist()
    # beams are distinct paths
    for b in range(3):
        paths = {tuple(out.beam_ids[b, w].tolist()) for w in range(W) if out.beam_cum[b, w] > -1e30}
        assert len(paths) == int((out.beam_cum[b] > -1e30).sum())


def test_fewer_expansions_than_width():
    _, lat, table, prev = _lattice(2, 10, 2, 50)
    out = _search(lat, table, prev, 16, 0.5)              # only 2, then 4 paths exist
    assert int((out.beam_cum[0] > -1e30).sum()) == 4
    assert (out.beam_ids[0, 4:] == -1).all() and torch.isinf(out.beam_score[0, 4:]).all()


def test_eos_early_stop_hand_built():
    V, L, K, eos = 16, 6, 3, 15
    x = torch.zeros((1, L, V))
    for i in range(L):
        x[0, i, i] = 5.0                                  # top-1 of position i is token i
        x[0, i, eos] = -9.0
    x[0, 2, eos] = 9.0                                    # EOS is top-1 at depth 3 (1-based)
    lat = oracle.lattice_build(x, K, eos_id=eos)
    table = torch.zeros((V, V))
    prev = torch.tensor([0], dtype=torch.int32)
    out = oracle.cps_search(lat.cand_id, lat.cand_logit, lat.lse64, lat.cand_count, prev, table,
                            W=4, lam=0.5, eos_id=eos, proxy_kind=1, V=V)
    assert out.path_len.item() == 3
    assert out.path[0].tolist() == [0, 1, eos, -1, -1, -1]
    assert out.row_status.item() & oracle.EOS_STOPPED
    assert lat.gen_len.item() == 2                        # Eq. 9 agrees: two positions before EOS
    # a lower-ranked beam placing EOS does not stop the search
    x[0, 2, eos] = 4.0                                    # now second at depth 3
    lat = oracle.lattice_build(x, K, eos_id=eos)
    out = oracle.cps_search(lat.cand_id, lat.cand_logit, lat.lse64, lat.cand_count, prev, table,
                            W=4, lam=0.5, eos_id=eos, proxy_kind=1, V=V)
    assert out.path_len.item() == L and out.path[0].tolist() == list(range(L))
    assert not out.row_status.item() & oracle.EOS_STOPPED


def test_proxy_changes_the_path_and_tie_break_is_lowest_id():
    V, L, K = 8, 2, 2
    x = torch.zeros((1, L, V))
    x[0, :, 3] = 1.0
    x[0, :, 5] = 1.0                                      # tokens 3 and 5 tie on the drafter's score
    lat = oracle.lattice_build(x, K)
    assert lat.cand_id[0, 0].tolist() == [3, 5]
    table = torch.zeros((V, V))
    prev = torch.tensor([0], dtype=torch.int32)
    out = oracle.cps_search(lat.cand_id, lat.cand_logit, lat.lse64, lat.cand_count, prev, table,
                            W=2, lam=0.5, proxy_kind=1, V=V)
    assert out.path[0].tolist() == [3, 3]                 # full tie: lowest ids
    table[3, 5] = 1.0                                     # the proxy prefers 3 -> 5
    out = oracle.cps_search(lat.cand_id, lat.cand_logit, lat.lse64, lat.cand_count, prev, table,
                            W=2, lam=0.5, proxy_kind=1, V=V)
    assert out.path[0].tolist() == [3, 5]


def test_hashed_proxy_index_follows_the_stated_mix():
    # the header text of the hashed table, restated with Python integers
    def idx(prev, cur, seed, log2):
        M = 0xFFFFFFFF
        h = (prev * 0x9E3779B1) & M
        h ^= (cur + seed) & M
        h = (h * 0x9E3779B1) & M
        h ^= h >> 15
        h = (h * 0x9E3779B1) & M
        h ^= h >> 13
        return h >> (32 - log2)
    log2 = 12
    table = torch.arange(1 << log2, dtype=torch.float32)   # score = its own index
    g = torch.Generator().manual_seed(0)
    hits = set()
    for prev, cur in torch.randint(0, 152064, (300, 2), generator=g).tolist():
        s = oracle.proxy_score(table, prev, cur, table_log2=log2, hash_seed=7)
        assert int(s) == idx(prev, cur, 7, log2)
        hits.add(int(s))
    assert len(hits) > 250                                 # spreads over the table


# ---- the richer causal proxies: a tensor of scores per (position, previous slot, slot), a hashed trigram ----
def _mix3(prev2, prev, cur, seed, log2):
    """The header text of the hashed trigram table, restated with Python integers."""
    M = 0xFFFFFFFF
    g = (prev2 * 0xC2B2AE35) & M
    g ^= g >> 16
    h = ((prev ^ g) * 0x9E3779B1) & M
    h ^= (cur + seed) & M
    h = (h * 0x9E3779B1) & M
    h ^= h >> 15
    h = (h * 0x9E3779B1) & M
    h ^= h >> 13
    return h >> (32 - log2)


def test_trigram_index_follows_the_stated_mix_and_uses_all_three_tokens():
    log2 = 14
    table = torch.arange(1 << log2, dtype=torch.float32)
    g = torch.Generator().manual_seed(1)
    for p2, p1, c in torch.randint(0, 152064, (300, 3), generator=g).tolist():
        assert int(oracle.trigram_score(table, p2, p1, c, table_log2=log2, hash_seed=3)) == _mix3(p2, p1, c, 3, log2)
    base = oracle.trigram_score(table, 5, 6, 7, table_log2=log2, hash_seed=3)
    others = [oracle.trigram_score(table, 9, 6, 7, table_log2=log2, hash_seed=3),
              oracle.trigram_score(table, 5, 9, 7, table_log2=log2, hash_seed=3),
              oracle.trigram_score(table, 5, 6, 9, table_log2=log2, hash_seed=3),
              oracle.trigram_score(table, 6, 5, 7, table_log2=log2, hash_seed=3)]
    assert all(o != base for o in others)


@pytest.mark.parametrize("kind", [2, 3])
@pytest.mark.parametrize("L,K,seed", [(3, 4, 0), (4, 3, 1), (5, 2, 2), (2, 5, 3)])
def test_wide_beam_equals_brute_force_with_tensor_and_trigram_proxies(kind, L, K, seed):
    V, lam, log2, hseed = 12, 0.4, 9, 11
    _, lat, _, _ = _lattice(L, V, K, seed)
    g = torch.Generator().manual_seed(100 + seed)
    KC = lat.cand_id.shape[2]
    if kind == 2:
        table = -6.0 * torch.rand((1, L, KC, KC), generator=g)
        prev = torch.tensor([4], dtype=torch.int32)
        ng = lambda i, ids, slots: float(table[0, i, 0 if i == 0 else slots[i - 1], slots[i]])
    else:
        table = -6.0 * torch.rand((1 << log2,), generator=g)
        prev = torch.tensor([[4, 9]], dtype=torch.int32)
        hist = lambda i, ids: ([4, 9] + list(ids))[i:i + 2]              # the two tokens before position i
        ng = lambda i, ids, slots: float(table[_mix3(hist(i, ids)[0], hist(i, ids)[1], ids[i], hseed, log2)])
    W = K ** (L - 1)
    out = oracle.cps_search(lat.cand_id, lat.cand_logit, lat.lse64, lat.cand_count, prev, table, W=W, lam=lam,
                            proxy_kind=kind, table_log2=log2, hash_seed=hseed, V=V)
    counts = lat.cand_count[0].tolist()
    scored = []
    for slots in itertools.product(*[range(c) for c in counts]):
        ids = [int(lat.cand_id[0, i, k]) for i, k in enumerate(slots)]
        s = sum(lam * (float(lat.cand_logit[0, i, k]) - float(lat.lse64[0, i])) + (1.0 - lam) * ng(i, ids, slots)
                for i, k in enumerate(slots))
        scored.append((s, ids))
    scored.sort(key=lambda t: -t[0])
    assert abs(out.path_score.item() - scored[0][0]) < 1e-4
    if scored[0][0] - scored[1][0] > 1e-4:
        assert out.path[0].tolist() == scored[0][1]
    nb = min(W, len(scored))
    assert np.allclose(out.beam_score[0, :nb].double().numpy(), np.array([s for s, _ in scored[:nb]]), atol=1e-4)


def test_tensor_proxy_built_from_the_dense_table_gives_the_dense_search():
    L, V, K, W, lam = 6, 30, 4, 3, 0.5
    _, lat, table, prev = _lattice(L, V, K, 9, B=2)
    dense = oracle.cps_search(lat.cand_id, lat.cand_logit, lat.lse64, lat.cand_count, prev, table, W=W, lam=lam,
                              proxy_kind=1, V=V)
    B, _, KC = lat.cand_id.shape
    tens = torch.zeros((B, L, KC, KC))
    for b in range(B):
        for i in range(L):
            for p in range(KC):
                pt = int(prev[b]) if i == 0 else int(lat.cand_id[b, i - 1, p])
                for k in range(KC):
                    ct = int(lat.cand_id[b, i, k])
                    if pt >= 0 and ct >= 0:
                        tens[b, i, p, k] = table[pt, ct]
    out = oracle.cps_search(lat.cand_id, lat.cand_logit, lat.lse64, lat.cand_count, prev, tens, W=W, lam=lam,
                            proxy_kind=2, V=V)
    for k in ("path", "path_slot", "path_len", "beam_ids", "beam_cum", "path_score", "beam_score"):
        assert torch.equal(getattr(out, k), getattr(dense, k)), k


# ---- verifier-aware scoring: a third term mu * l^ver(position, slot) in Eq. 8 ----
@pytest.mark.parametrize("L,K,seed,mu", [(3, 4, 10, 0.7), (4, 3, 11, 1.5), (5, 2, 12, 0.25)])
def test_verifier_term_wide_beam_equals_brute_force(L, K, seed, mu):
    V, lam = 12, 0.5
    _, lat, table, prev = _lattice(L, V, K, seed)
    g = torch.Generator().manual_seed(seed + 100)
    ver = -5.0 * torch.rand((1, L, K), generator=g)
    W = K ** (L - 1)
    out = oracle.cps_search(lat.cand_id, lat.cand_logit, lat.lse64, lat.cand_count, prev, table, W=W, lam=lam,
                            proxy_kind=1, V=V, ver_score=ver, mu=mu)
    scored = []
    for slots in itertools.product(*[range(c) for c in lat.cand_count[0].tolist()]):
        ids = [int(lat.cand_id[0, i, k]) for i, k in enumerate(slots)]
        s = _eq8(lat, table, prev, 0, ids, slots, lam) + mu * sum(float(ver[0, i, k]) for i, k in enumerate(slots))
        scored.append((s, ids))
    scored.sort(key=lambda t: -t[0])
    assert abs(out.path_score.item() - scored[0][0]) < 1e-4
    if scored[0][0] - scored[1][0] > 1e-4:
        assert out.path[0].tolist() == scored[0][1]
    nb = min(W, len(scored))
    assert np.allclose(out.beam_score[0, :nb].double().numpy(), np.array([s for s, _ in scored[:nb]]), atol=1e-4)


def test_verifier_term_limits():
    V, L, K, lam = 20, 6, 4, 0.5
    _, lat, table, prev = _lattice(L, V, K, 21, B=3)
    g = torch.Generator().manual_seed(5)
    ver = -4.0 * torch.rand((3, L, K), generator=g)
    kw = dict(W=3, lam=lam, proxy_kind=1, V=V)
    base = oracle.cps_search(lat.cand_id, lat.cand_logit, lat.lse64, lat.cand_count, prev, table, **kw)
    zero = oracle.cps_search(lat.cand_id, lat.cand_logit, lat.lse64, lat.cand_count, prev, table, ver_score=ver, mu=0.0, **kw)
    for f in ("path", "path_len", "beam_ids", "beam_cum", "path_score"):       # mu = 0: Eq. 8 as it is, bit for bit
        assert torch.equal(getattr(base, f), getattr(zero, f)), f
    big = oracle.cps_search(lat.cand_id, lat.cand_logit, lat.lse64, lat.cand_count, prev, table, ver_score=ver, mu=1e4, **kw)
    want = torch.gather(lat.cand_id, 2, ver.argmax(dim=2, keepdim=True)).squeeze(2)   # the verifier's favourite everywhere
    assert torch.equal(big.path, want)
    const = oracle.cps_search(lat.cand_id, lat.cand_logit, lat.lse64, lat.cand_count, prev, table,
                              ver_score=torch.full((3, L, K), -2.0), mu=0.5, **kw)
    assert torch.equal(const.path, base.path)                                   # a constant shifts every path alike
    assert torch.allclose(const.path_score, base.path_score - 0.5 * 2.0 * L, atol=1e-4)
