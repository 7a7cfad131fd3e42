"""Seeded stand-in for a draft model's proposals in the draft-then-verify loop.

A randomly initialised draft model cannot predict a randomly initialised target, so the proposals are the
target's own greedy transcript (computed beforehand by whoever builds the workload), each position independently
replaced by a uniform token with probability `corrupt_p`.  Per round the proposer draws a draft length
(adaptive-length drafting, Section IV-A), reuses the part of the previous draft that lies beyond the rejection
point as the head of the new trunk (a simplified form of draft sequence recycling, Section IV-B), hangs short
side branches of uniform tokens off the trunk (sparse tree, Section IV-C) and says which tokens the draft model
has to be stepped on to produce the new part of the trunk.  No decoder arithmetic here.
"""
import numpy as np

from .trees import fill_tree_tokens, trunk_tree

_STREAM_PROPOSE = 0x9A05


class CorruptedGreedyProposer:
    def __init__(self, transcripts, roots, vocab, seed=0, n_nodes=32, k_min=4, k_max=16, corrupt_p=0.2):
        self.T = [list(map(int, t)) for t in transcripts]
        self.roots = [int(r) for r in roots]
        self.vocab, self.seed, self.n_nodes = int(vocab), int(seed), int(n_nodes)
        self.k_min, self.k_max, self.p = int(k_min), int(k_max), float(corrupt_p)
        self.round = [0] * len(self.T)
        self.tail = [[] for _ in self.T]          # recycled proposals: tail[b][i] proposes T[b][emitted + i]
        self.trunk = [[] for _ in self.T]

    def propose(self, b, emitted):
        """Returns (tokens, parent, draft_feed) for utterance b given the tokens it has emitted so far."""
        e = len(emitted)
        rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence(
            entropy=[self.seed, _STREAM_PROPOSE, b, self.round[b]])))
        k = int(rng.integers(self.k_min, self.k_max + 1))
        k = min(k, self.n_nodes - 1, len(self.T[b]) - e)
        if k < 1:
            raise ValueError("transcript too short for another round")
        trunk = list(self.tail[b][:k])
        for pos in range(e + len(trunk), e + k):
            tok = self.T[b][pos]
            if rng.random() < self.p:
                tok = int(rng.integers(0, self.vocab))
            trunk.append(tok)
        root = emitted[-1] if e else self.roots[b]
        parent = trunk_tree(self.n_nodes, k, seed=self.seed * 1000003 + b * 1009 + self.round[b])
        tokens = fill_tree_tokens(parent, self.vocab, seed=self.seed * 7919 + b * 104729 + self.round[b],
                                  root_token=root, main_tokens=trunk)
        n_recycled = min(len(self.tail[b]), k)
        feed = ([root] + trunk)[n_recycled:k]      # one draft step per new trunk token
        self.trunk[b] = trunk
        self.round[b] += 1
        return tokens, parent, feed

    def observe(self, b, accept_len):
        """The outcome of the verification: proposals beyond the rejected one stay valid for the positions they were
        drafted for and head the next trunk."""
        self.tail[b] = self.trunk[b][accept_len + 1:]
