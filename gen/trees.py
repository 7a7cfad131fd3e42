"""Seeded draft-token-tree topologies and token fills.

A tree is `parent[n]` (int32) with parent[0] = -1 and parent[i] < i; node 0 is
the root (the last committed token), the other nodes are draft tokens.  The
shapes imitate the paper's drafts: plain chains (single-sequence prediction,
Section IV-A), and a long trunk with a few short side branches (two-pass
sparse-tree prediction, Section IV-C).
"""
import numpy as np

_STREAM_TREE = 0x73EE
_STREAM_FILL = 0xF111
_STREAM_CORRUPT = 0xC033
_STREAM_RELABEL = 0x3E1A


def _rng(seed: int, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence(entropy=[int(seed), stream])))


def chain_tree(k_drafts: int) -> np.ndarray:
    """Root followed by a linear chain of k draft nodes (n = k + 1)."""
    return np.arange(-1, k_drafts, dtype=np.int32)


def complete_binary_tree(n_nodes: int) -> np.ndarray:
    """Breadth-first numbered binary tree: parent[i] = (i - 1) // 2."""
    p = (np.arange(n_nodes, dtype=np.int64) - 1) // 2
    p[0] = -1
    return p.astype(np.int32)


def sparse_tree(n_nodes: int, seed: int = 0, root_fanout: int = 4, level2_fanout: int = 2,
                levels: int | None = None) -> np.ndarray:
    """Root with `root_fanout` children, each of those with `level2_fanout` children, then chains.

    The first chain (below the first grandchild) is the main trunk.  With `levels` given the
    trunk reaches exactly that many levels counting the root and no other chain is longer; the
    remaining nodes are spread over the other chains by a seeded multinomial draw.  Without it the
    trunk takes half of the chain nodes.  Nodes are numbered level by level for the bushy top and
    chain by chain afterwards, so parent[i] < i always holds.
    """
    rng = _rng(seed, _STREAM_TREE)
    parent = [-1]
    level2 = []
    for _ in range(root_fanout):
        if len(parent) >= n_nodes:
            break
        level2.append(len(parent))
        parent.append(0)
    level3 = []
    for p in level2:
        for _ in range(level2_fanout):
            if len(parent) >= n_nodes:
                break
            level3.append(len(parent))
            parent.append(p)
    rest = n_nodes - len(parent)
    if rest > 0:
        n_chains = len(level3)
        if levels is not None:
            cap = levels - 3
            if cap < 0 or cap * n_chains < rest or rest < cap:
                raise ValueError("levels incompatible with n_nodes")
            main_len = cap
        else:
            cap = rest
            main_len = (rest + 1) // 2 if n_chains > 1 else rest
        lens = np.zeros(n_chains, dtype=np.int64)
        lens[0] = main_len
        left = rest - main_len
        while left > 0:
            open_chains = [c for c in range(1, n_chains) if lens[c] < cap]
            c = open_chains[int(rng.integers(0, len(open_chains)))]
            lens[c] += 1
            left -= 1
        for c in range(n_chains):
            prev = level3[c]
            for _ in range(int(lens[c])):
                parent.append(prev)
                prev = len(parent) - 1
    return np.asarray(parent, dtype=np.int32)


def trunk_tree(n_nodes: int, trunk_len: int, seed: int = 0, max_branch: int = 3) -> np.ndarray:
    """Root, a trunk (chain) of `trunk_len` draft nodes numbered 1..trunk_len, and the remaining nodes as short
    side branches: each is a chain of 1..max_branch nodes hanging off a seeded trunk node (or the root) as a
    sibling of the next trunk node -- the long-trunk / few-short-branches shape of a sparse draft tree
    (Section IV-C).  The trunk is the main path (its nodes are the lowest-numbered children)."""
    if trunk_len < 1 or trunk_len + 1 > n_nodes:
        raise ValueError("trunk does not fit")
    rng = _rng(seed, _STREAM_TREE)
    parent = [-1] + list(range(trunk_len))
    while len(parent) < n_nodes:
        length = int(min(rng.integers(1, max_branch + 1), n_nodes - len(parent)))
        prev = int(rng.integers(0, trunk_len))          # branches off below trunk node `prev` (0 = root)
        for _ in range(length):
            parent.append(prev)
            prev = len(parent) - 1
    return np.asarray(parent, dtype=np.int32)


def main_path(parent: np.ndarray) -> np.ndarray:
    """Node indices root -> leaf obtained by always stepping to the lowest-numbered child."""
    n = len(parent)
    first_child = np.full(n, -1, dtype=np.int64)
    for i in range(n - 1, 0, -1):
        first_child[parent[i]] = i
    path = [0]
    while first_child[path[-1]] >= 0:
        path.append(int(first_child[path[-1]]))
    return np.asarray(path, dtype=np.int32)


def fill_tree_tokens(parent: np.ndarray, vocab: int, seed: int, root_token: int,
                     main_tokens=None, corrupt_p: float = 0.0) -> np.ndarray:
    """Tokens for every node.

    All nodes draw uniformly; the root gets `root_token`; if `main_tokens` is given, the j-th node
    after the root on the main path gets main_tokens[j-1], each position independently replaced by
    a uniform token with probability `corrupt_p`.  Side nodes are redrawn until no two children of
    one parent carry the same token.
    """
    n = len(parent)
    rng = _rng(seed, _STREAM_FILL)
    tokens = rng.integers(0, vocab, size=n, dtype=np.int32)
    tokens[0] = root_token
    fixed = np.zeros(n, dtype=bool)
    fixed[0] = True
    if main_tokens is not None:
        crng = _rng(seed, _STREAM_CORRUPT)
        path = main_path(parent)[1:]
        k = min(len(path), len(main_tokens))
        flips = crng.random(k) < corrupt_p
        repl = crng.integers(0, vocab, size=k, dtype=np.int32)
        for j in range(k):
            tokens[path[j]] = repl[j] if flips[j] else main_tokens[j]
            fixed[path[j]] = True
    for i in range(1, n):
        if fixed[i]:
            continue
        sibs = [j for j in range(1, n) if parent[j] == parent[i] and j != i and (fixed[j] or j < i)]
        while any(tokens[j] == tokens[i] for j in sibs):
            tokens[i] = rng.integers(0, vocab, dtype=np.int32)
    return tokens


def relabel_tree(parent: np.ndarray, tokens: np.ndarray, seed: int):
    """A random renumbering that keeps parent[i] < i.  Returns (parent', tokens', old_of_new)."""
    n = len(parent)
    rng = _rng(seed, _STREAM_RELABEL)
    placed = [0]
    ready = [i for i in range(1, n) if parent[i] == 0]
    while ready:
        pick = ready.pop(int(rng.integers(0, len(ready))))
        placed.append(pick)
        ready += [i for i in range(1, n) if parent[i] == pick]
    old_of_new = np.asarray(placed, dtype=np.int32)
    new_of_old = np.empty(n, dtype=np.int32)
    new_of_old[old_of_new] = np.arange(n, dtype=np.int32)
    new_parent = np.array([-1 if parent[o] < 0 else new_of_old[parent[o]] for o in old_of_new], dtype=np.int32)
    return new_parent, np.asarray(tokens)[old_of_new].astype(np.int32), old_of_new
