import numpy as np
import torch

import gen


def test_bf16_rounding_matches_library_rne():
    rng = np.random.default_rng(1)
    x = np.concatenate([rng.standard_normal(4096).astype(np.float32) * 0.02,
                        np.array([0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.0e38, 1e-40], np.float32)])
    bits = gen.f32_to_bf16_bits(x)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(bits, ref)
    back = gen.bf16_bits_to_f32(bits)
    assert np.array_equal(back, torch.from_numpy(x).to(torch.bfloat16).float().numpy())


def test_weights_are_reproducible_and_random_access():
    cfg = gen.get_config("micro")
    a = gen.WeightStore(cfg, 3)
    b = gen.WeightStore(cfg, 3)
    assert np.array_equal(a.tensor(1, "wd"), b.layer(1)["wd"])
    assert not np.array_equal(a.tensor(0, "wq"), a.tensor(1, "wq"))
    assert not np.array_equal(a.tensor(0, "wq"), gen.WeightStore(cfg, 4).tensor(0, "wq"))
    w = gen.bf16_bits_to_f32(a.tensor(0, "wg"))
    assert w.shape == (cfg.ffn, cfg.d_model)
    assert abs(w.std() - 0.02) < 2e-3
    g = a.tensor(0, "g_attn")
    assert g.dtype == np.float32 and abs(g.mean() - 1.0) < 0.01
    seen = {}
    a.map_tensors(lambda l, n, arr: seen.__setitem__((l, n), arr.shape), a.all_keys(), threads=3)
    assert len(seen) == 3 + 9 * cfg.n_layers


def test_tree_generators():
    p = gen.sparse_tree(64, seed=0, levels=12)
    assert len(p) == 64 and p[0] == -1 and all(0 <= p[i] < i for i in range(1, 64))
    assert list(p[1:5]) == [0, 0, 0, 0] and list(p[5:13]) == [1, 1, 2, 2, 3, 3, 4, 4]
    depth = np.zeros(64, int)
    for i in range(1, 64):
        depth[i] = depth[p[i]] + 1
    assert depth.max() == 11                       # 12 levels counting the root
    mp = gen.main_path(p)
    assert len(mp) == 12 and list(depth[mp]) == list(range(12))
    for n in (16, 256):
        q = gen.sparse_tree(n, seed=1)
        assert len(q) == n and all(0 <= q[i] < i for i in range(1, n))
    assert list(gen.chain_tree(3)) == [-1, 0, 1, 2]
    assert list(gen.complete_binary_tree(7)) == [-1, 0, 0, 1, 1, 2, 2]
    toks = gen.fill_tree_tokens(p, 50, seed=2, root_token=7, main_tokens=list(range(100, 111)), corrupt_p=0.0)
    assert toks[0] == 7 and list(toks[mp[1:]]) == list(range(100, 111))
    for i in range(64):
        kids = [int(toks[j]) for j in range(1, 64) if p[j] == i]
        assert len(kids) == len(set(kids))
    p2, t2, old = gen.relabel_tree(p, toks, seed=5)
    assert all(0 <= p2[i] < i for i in range(1, 64)) and sorted(old) == list(range(64))
    for new in range(1, 64):
        assert old[p2[new]] == p[old[new]] and t2[new] == toks[old[new]]


def test_trunk_tree_and_proposer_follow_their_contracts():
    """trunk_tree: the trunk is the main path and parents precede children; the proposer replays a transcript with
    seeded corruption, recycles the tail past a rejection and asks for one draft step per new trunk token."""
    for n, k, seed in ((32, 4, 0), (32, 16, 1), (12, 11, 2), (2, 1, 3)):
        parent = gen.trunk_tree(n, k, seed=seed)
        assert len(parent) == n and parent[0] == -1 and all(0 <= parent[i] < i for i in range(1, n))
        assert list(gen.main_path(parent)) == list(range(k + 1))
        assert np.array_equal(parent, gen.trunk_tree(n, k, seed=seed))
    rng = np.random.default_rng(3)
    T = [list(rng.integers(0, 1000, 120)), list(rng.integers(0, 1000, 120))]
    roots = [7, 9]
    P = gen.CorruptedGreedyProposer(T, roots, 1000, seed=4, n_nodes=32, k_min=4, k_max=16, corrupt_p=0.2)
    Q = gen.CorruptedGreedyProposer(T, roots, 1000, seed=4, n_nodes=32, k_min=4, k_max=16, corrupt_p=0.2)
    for b in range(2):
        emitted, steps, drafted = [], 0, 0
        prev_trunk, prev_a = None, None
        while len(emitted) < 80:
            tokens, parent, feed = P.propose(b, emitted)
            t2, p2, f2 = Q.propose(b, emitted)
            assert np.array_equal(tokens, t2) and np.array_equal(parent, p2) and list(feed) == list(f2)   # seeded
            k = len(gen.main_path(parent)) - 1
            assert 1 <= k <= 16 and len(tokens) == 32 and tokens[0] == (emitted[-1] if emitted else roots[b])
            trunk = [int(x) for x in tokens[1:k + 1]]
            if prev_trunk is not None:
                tail = prev_trunk[prev_a + 1:][:k]
                assert trunk[:len(tail)] == tail                        # recycled proposals head the new trunk
                assert len(feed) == k - len(tail)                       # one draft step per new token
                assert list(feed) == ([int(tokens[0])] + trunk)[len(tail):k]
            else:
                assert len(feed) == k
            # siblings carry different tokens
            for i in range(1, 32):
                assert all(tokens[i] != tokens[j] for j in range(1, 32) if j != i and parent[j] == parent[i])
            a = 0
            while a < k and trunk[a] == T[b][len(emitted) + a]:
                a += 1
            emitted += trunk[:a] + [T[b][len(emitted) + a]]
            P.observe(b, a)
            Q.observe(b, a)
            prev_trunk, prev_a = trunk, a
            steps += 1
            drafted += len(feed)
        assert emitted == T[b][:len(emitted)]
        assert steps < 40 and drafted < sum(1 for _ in emitted) * 4
