"""Host controller of the draft-then-verify loop (Section II-B, Fig. 3) for a batch of concurrent utterances.

Control flow only: every forward pass, the accept rule and the cache compaction run in the library's kernels
(specasr_verify_tree_batch / specasr_commit_kv / specasr_kv_truncate).  Per round the controller
  1. asks the caller's proposer for each utterance's draft tree and for the tokens the draft model is to be
     stepped on (the proposer decides draft length, recycling of an earlier draft's tail, tree shape),
  2. steps the draft model autoregressively, all utterances in one batched single-node call per step,
  3. verifies all trees in one batched call of the target model and commits every utterance's accepted path,
  4. reads accept lengths, paths and bonus tokens back (the one host synchronisation of a round) and appends
     the accepted draft tokens and the bonus token to each transcript.
"""
import numpy as np
import torch

from . import binding as B
from .runtime import BatchVerifier, DeviceKV


class SpeculativeBatchLoop:
    def __init__(self, target_kvs, draft_kvs=None):
        """target_kvs: one DeviceKV per utterance (prefix already filled); the first one's workspace must hold
        the nodes of all trees of a round.  draft_kvs: the draft model's caches (same order), or None to skip
        the draft phase."""
        self.target_kvs = list(target_kvs)
        self.draft_kvs = list(draft_kvs) if draft_kvs is not None else None
        self.B = len(self.target_kvs)
        self.device = self.target_kvs[0].model.device
        self._verifiers = {}
        self.target_len = [kv.length() for kv in self.target_kvs]
        if self.draft_kvs is not None:
            self.draft_len = [kv.length() for kv in self.draft_kvs]     # entries that match the committed text
            self.draft_dev_len = list(self.draft_len)                   # entries the device cache holds
            self._minus_one = torch.full((self.B,), -1, dtype=torch.int32, device=self.device)
        self.rounds = 0               # batched verification calls
        self.utterance_rounds = 0     # trees verified (rounds summed over utterances)
        self.draft_steps = 0          # batched draft-model calls

    # ---- draft phase -----------------------------------------------------------------------------------------
    def _verifier(self, kvs, members):
        """Output buffers for one subset of the utterances (utterances leave the batch as they finish)."""
        key = (id(kvs), tuple(members))
        if key not in self._verifiers:
            self._verifiers[key] = BatchVerifier([kvs[b] for b in members])
        return self._verifiers[key]

    def run_draft(self, feeds, missing=None):
        """feeds: {b: tokens} -- tokens the draft model of utterance b consumes this round, one per autoregressive step.
        Step j runs every utterance that still has a token left as one batched call of single-node trees and
        appends that token's K/V to its draft cache.  (The proposer supplies the draft tokens, so the draft
        model's own arg-max is not read back.)  missing: {b: committed tokens the draft cache has not seen yet}
        (pending_alignment); they ride in front of the utterance's first token as one chain, all utterances in the
        same batched call, instead of one call per utterance before the round."""
        if self.draft_kvs is None:
            return
        missing = missing or {}
        steps = max((len(f) for f in feeds.values()), default=0)
        if any(len(m) > 0 for m in missing.values()):
            steps = max(steps, 1)
        for j in range(steps):
            if j == 0:
                chains = {b: [int(t) for t in missing.get(b, [])] + [int(t) for t in feeds[b][:1]] for b in sorted(feeds)}
                members = [b for b in sorted(feeds) if chains[b]]
            else:
                chains = {b: [int(feeds[b][j])] for b in sorted(feeds) if len(feeds[b]) > j}
                members = sorted(chains)
            if not members:
                continue
            bv = self._verifier(self.draft_kvs, members)
            sizes = [len(chains[b]) for b in members]
            if max(sizes) == 1:
                toks = torch.tensor([chains[b][0] for b in members], dtype=torch.int32, device=self.device)
                bv.verify(toks, self._minus_one[:len(members)], list(range(len(members) + 1)))
                bv.commit()
            else:
                toks = torch.tensor([t for b in members for t in chains[b]], dtype=torch.int32, device=self.device)
                par = torch.tensor([i - 1 for n in sizes for i in range(n)], dtype=torch.int32, device=self.device)
                bv.verify(toks, par, [0] + list(np.cumsum(sizes)))
                bv.commit_chains()
            for b, n in zip(members, sizes):
                self.draft_len[b] += n
                self.draft_dev_len[b] += n
            self.draft_steps += 1

    def pending_alignment(self, b, committed_tokens):
        """As align_draft, but the committed tokens the draft cache has not seen are returned (for run_draft to put in
        front of the utterance's first draft token) instead of being fed in a call of their own."""
        if self.draft_kvs is None:
            return []
        want = self.target_len[b]
        have = min(self.draft_len[b], want)
        if self.draft_dev_len[b] != have:
            self.draft_kvs[b].truncate(have)
        self.draft_len[b] = self.draft_dev_len[b] = have
        if have == want:
            return []
        return [int(t) for t in committed_tokens[len(committed_tokens) - 1 - (want - have):len(committed_tokens) - 1]]

    def align_draft(self, b, committed_tokens):
        """Brings utterance b's draft cache to the target's committed length (everything but the next root, which
        neither cache holds yet): drops draft entries past it, or feeds the committed tokens it has not seen as
        one chain.  committed_tokens ends with the next root."""
        if self.draft_kvs is None:
            return
        want = self.target_len[b]
        kv = self.draft_kvs[b]
        have = min(self.draft_len[b], want)
        if self.draft_dev_len[b] != have:
            kv.truncate(have)
        if have < want:
            missing = committed_tokens[len(committed_tokens) - 1 - (want - have):len(committed_tokens) - 1]
            kv.prefill_tokens(torch.tensor([int(t) for t in missing], dtype=torch.int32, device=self.device))
        self.draft_len[b] = self.draft_dev_len[b] = want

    # ---- verification ----------------------------------------------------------------------------------------
    def verify_round(self, trees):
        """trees: {b: (tokens, parent)} int32 arrays for the utterances still decoding.  Returns
        {b: (accept_len, path, bonus)} as host values after committing each of them."""
        members = sorted(trees)
        offsets = np.concatenate([[0], np.cumsum([len(trees[b][0]) for b in members])]).astype(int)
        tokens = torch.from_numpy(np.concatenate([np.asarray(trees[b][0], np.int32) for b in members])).to(self.device)
        parent = torch.from_numpy(np.concatenate([np.asarray(trees[b][1], np.int32) for b in members])).to(self.device)
        bv = self._verifier(self.target_kvs, members)
        bv.verify(tokens, parent, offsets)
        bv.commit()
        accept = bv.out_accept.cpu().numpy()           # synchronises the stream
        path = bv.out_path[:offsets[-1]].cpu().numpy()
        bonus = bv.out_bonus.cpu().numpy()
        out = {}
        for i, b in enumerate(members):
            a = int(accept[i])
            if a < 0:
                raise RuntimeError(f"verification of utterance {b} failed on the device "
                                   f"(status {self.target_kvs[b].status()})")
            self.target_len[b] += a + 1
            out[b] = (a, path[offsets[i]:offsets[i] + a + 1].copy(), int(bonus[i]))
        self.rounds += 1
        self.utterance_rounds += len(members)
        return out

    # ---- the loop --------------------------------------------------------------------------------------------
    def decode(self, roots, n_tokens, proposer):
        """Runs rounds until every utterance has emitted n_tokens tokens; an utterance leaves the batch when it
        has.  roots[b] is the last committed token of
        utterance b (the root of its first tree); draft and target caches must start at equal lengths.  `proposer.propose(b, emitted)` returns (tokens, parent,
        draft_feed) for the next round of utterance b.  Returns the transcripts (lists of token ids)."""
        emitted = [[] for _ in range(self.B)]
        history = [[int(r)] for r in roots]            # committed tokens ending with the current root
        while True:
            active = [b for b in range(self.B) if len(emitted[b]) < n_tokens]
            if not active:
                break
            trees, feeds, missing = {}, {}, {}
            for b in active:
                tokens, parent, feed = proposer.propose(b, emitted[b])
                assert int(tokens[0]) == history[b][-1]
                trees[b] = (tokens, parent)
                feeds[b] = feed
                missing[b] = self.pending_alignment(b, history[b])
            self.run_draft(feeds, missing)
            for b, (a, path, bonus) in self.verify_round(trees).items():
                accepted = [int(trees[b][0][i]) for i in path[1:]]
                emitted[b] += accepted + [bonus]
                history[b] += accepted + [bonus]
                proposer.observe(b, a)
        return [e[:n_tokens] for e in emitted]

    # ---- drafts from the draft model itself ------------------------------------------------------------------
    def draft_trees(self, members, roots, threshold, max_len):
        """Greedy single-sequence drafting with the draft model for the utterances in `members` (all of them in
        one batched single-node call per step).  After every step the top-2 tokens and their softmax
        probabilities are read back: the top-1 token extends the trunk; where its probability is below
        `threshold` the second-ranked token becomes a one-node side branch at that position and the utterance
        stops drafting (adaptive truncation, Section IV-A, with the limited-width expansion of Section IV-C at
        the point of uncertainty); nobody drafts more than `max_len` tokens.  Returns {b: (tokens, parent)}."""
        trunk = {b: [] for b in members}
        branch = {b: None for b in members}            # (depth of the parent on the trunk, token)
        cur = {b: int(roots[b]) for b in members}
        live = list(members)
        for _ in range(max_len):
            if not live:
                break
            bv = self._verifier(self.draft_kvs, live)
            nb = len(live)
            toks = torch.tensor([cur[b] for b in live], dtype=torch.int32, device=self.device)
            # top-2 tokens and probabilities come out of the vocabulary projection's epilogue: no logits matrix is written
            bv.verify_top2(toks, self._minus_one[:nb], list(range(nb + 1)))
            bv.commit()
            bv.top_ids, bv.top_probs = bv.out_top2_ids[:nb], bv.out_top2_probs[:nb]
            ids = bv.top_ids.cpu().numpy()             # synchronises: the host decides who goes on
            probs = bv.top_probs.cpu().numpy()
            self.draft_steps += 1
            still = []
            for i, b in enumerate(live):
                self.draft_len[b] += 1
                self.draft_dev_len[b] += 1
                trunk[b].append(int(ids[i, 0]))
                cur[b] = int(ids[i, 0])
                if probs[i, 0] < threshold:
                    branch[b] = (len(trunk[b]) - 1, int(ids[i, 1]))
                else:
                    still.append(b)
            live = still
        trees = {}
        for b in members:
            k = len(trunk[b])
            tokens = [int(roots[b])] + trunk[b]
            parent = [-1] + list(range(k))
            if branch[b] is not None and branch[b][1] != trunk[b][branch[b][0]]:
                parent.append(branch[b][0])            # sibling of trunk node depth + 1
                tokens.append(branch[b][1])
            trees[b] = (np.asarray(tokens, np.int32), np.asarray(parent, np.int32))
        return trees

    def decode_with_draft_model(self, roots, n_tokens, threshold=0.4, max_len=24):
        """The loop with the draft model's own proposals (no stand-in): rounds of draft_trees -> batched
        verification -> commit until every utterance has emitted n_tokens tokens."""
        if self.draft_kvs is None:
            raise ValueError("no draft caches were given")
        emitted = [[] for _ in range(self.B)]
        history = [[int(r)] for r in roots]
        while True:
            active = [b for b in range(self.B) if len(emitted[b]) < n_tokens]
            if not active:
                break
            for b in active:
                self.align_draft(b, history[b])
            start = {b: self.draft_len[b] for b in active}
            trees = self.draft_trees(active, {b: history[b][-1] for b in active}, threshold, max_len)
            for b, (a, path, bonus) in self.verify_round(trees).items():
                tokens = trees[b][0]
                accepted = [int(tokens[i]) for i in path[1:]]
                emitted[b] += accepted + [bonus]
                history[b] += accepted + [bonus]
                # the draft cache holds the root and the trunk tokens it was stepped on: keep what the target kept
                on_trunk = 0
                while on_trunk < a and int(path[on_trunk + 1]) == on_trunk + 1:
                    on_trunk += 1
                self.draft_len[b] = min(self.draft_len[b], start[b] + on_trunk + 1)
        return [e[:n_tokens] for e in emitted]

    def decode_with_strategies(self, roots, n_tokens, strategy="two_pass", threshold=0.4, max_len=24, n_nodes=32,
                               max_branch=4, max_regen=6):
        """The whole method (Fig. 7): per round every utterance drafts with the draft model -- `two_pass`: a
        two-pass sparse tree (Section IV-C); `recycle`: a single sequence that starts from the recycled remains of
        the previous draft (Section IV-B) and is extended greedily until a token falls below the threshold or
        max_len is reached (Section IV-A) -- then all trees are verified by the target in one batched call and the
        accepted paths are committed.  Returns the transcripts.  `self.draft_forwards` counts draft-model passes."""
        if self.draft_kvs is None:
            raise ValueError("no draft caches were given")
        emitted = [[] for _ in range(self.B)]
        history = [[int(r)] for r in roots]
        last = [None] * self.B                               # (trunk tokens, accept_len, last accepted token) of the last round
        strategies = [DraftStrategies(kv) for kv in self.draft_kvs]
        while True:
            active = [b for b in range(self.B) if len(emitted[b]) < n_tokens]
            if not active:
                break
            trees = {}
            for b in active:
                self.align_draft(b, history[b])              # the draft cache holds everything before the root
                ds, root = strategies[b], history[b][-1]
                if strategy == "two_pass":
                    t = ds.two_pass_tree(root, max_len, threshold, n_nodes, max_branch)
                    trees[b] = (t["tokens"], t["parent"])
                    continue
                trunk = []
                if last[b] is not None and last[b][1] < len(last[b][0]):
                    old, a, kept = last[b]
                    kv = self.draft_kvs[b]
                    kv.truncate(self.target_len[b] - 1)      # recycling decodes under the last accepted token
                    trunk = ds.recycled_draft(kept, old, a, root, max_len, max_regen)["draft"]
                    kv.prefill_tokens(torch.tensor([kept], dtype=torch.int32, device=self.device))
                path = [root] + trunk                        # extend what was recycled, adaptively
                while len(trunk) < max_len:
                    ids, probs = ds._chain_top2(path)
                    trunk.append(int(ids[0]))
                    path.append(int(ids[0]))
                    if probs[0] < threshold:
                        break
                trees[b] = (np.asarray([root] + trunk, np.int32), np.arange(-1, len(trunk), dtype=np.int32))
            for b, (a, path, bonus) in self.verify_round(trees).items():
                tokens = trees[b][0]
                accepted = [int(tokens[i]) for i in path[1:]]
                kept = accepted[-1] if accepted else history[b][-1]
                emitted[b] += accepted + [bonus]
                history[b] += accepted + [bonus]
                last[b] = ([int(t) for t in tokens[1:]], a, kept) if strategy == "recycle" else None
        self.draft_forwards = sum(ds.forwards for ds in strategies)
        return [e[:n_tokens] for e in emitted]


# ---------------------------------------------------------------------------------------------------------------
# Drafting strategies of Section IV on the draft model.  Control flow only: every forward pass of the draft model is
# one tree-verification call of the library on the draft cache (the tree-masked attention is what lets two sequences
# be decoded side by side, Section IV-B), and the top-2 tokens / probabilities come out of the vocabulary
# projection's epilogue (specasr_verify_tree_top2).  A step re-verifies the whole uncommitted tree from its root, so
# the draft cache itself is never advanced or rewound while drafting.

RECYCLE_OFFSETS = (0, -1, 1)            # "corresponding or adjacent positions" (Section IV-B)


def match_position(seq_tokens, seq_first_pos, token, pos, lowest_pos=None):
    """Index into seq_tokens (whose first token sits at position seq_first_pos) of the first position among pos,
    pos - 1, pos + 1 at which it carries `token`, or None."""
    for off in RECYCLE_OFFSETS:
        q = pos + off
        if lowest_pos is not None and q < lowest_pos:
            continue
        i = q - seq_first_pos
        if 0 <= i < len(seq_tokens) and int(seq_tokens[i]) == int(token):
            return i
    return None


class DraftStrategies:
    """The draft side of one utterance.  `draft_kv` holds the context up to, not including, node 0 of the trees
    passed to it (the usual convention: the root's K/V is not in the cache yet)."""

    def __init__(self, draft_kv: DeviceKV):
        self.kv = draft_kv
        self.device = draft_kv.model.device
        self.forwards = 0

    def tree_top2(self, tokens, parent):
        """One forward pass of the draft model over a token tree: (ids [n, 2], probs [n, 2]) on the host."""
        t = torch.tensor([int(x) for x in tokens], dtype=torch.int32, device=self.device)
        p = torch.tensor([int(x) for x in parent], dtype=torch.int32, device=self.device)
        self.kv.verify_top2(t, p)
        self.forwards += 1
        n = len(tokens)
        ids = self.kv.out_top2_ids[:n].cpu().numpy()           # synchronises: the host decides how to go on
        probs = self.kv.out_top2_probs[:n].cpu().numpy()
        if int(ids[0, 0]) < 0:
            raise RuntimeError(f"draft forward failed on the device (status {self.kv.status()})")
        return ids, probs

    def _chain_top2(self, path):
        ids, probs = self.tree_top2(path, [-1] + list(range(len(path) - 1)))
        return ids[-1], probs[-1]

    def adaptive_sequence(self, root, max_len, threshold):
        """Section IV-A: greedy drafting that stops after the first token whose probability is below the threshold."""
        path, out = [int(root)], []
        for _ in range(max_len):
            ids, probs = self._chain_top2(path)
            out.append(int(ids[0]))
            path.append(int(ids[0]))
            if probs[0] < threshold:
                break
        return out

    def two_pass_tree(self, root, max_len, threshold, n_nodes, max_branch):
        """Section IV-C: trunk by greedy decoding with uncertain positions marked, then one branch per mark that
        starts with the second-ranked token and ends where it meets the trunk or an earlier branch."""
        tokens, parent, depth = [int(root)], [-1], [0]
        marks = []
        for j in range(1, max_len + 1):
            if len(tokens) >= n_nodes:
                break
            ids, probs = self._chain_top2(tokens)              # the trunk so far is a chain
            tokens.append(int(ids[0]))
            parent.append(len(tokens) - 2)
            depth.append(j)
            if probs[0] < threshold and int(ids[1]) != int(ids[0]):
                marks.append((j, int(ids[1])))
        m = len(tokens) - 1
        grown = []

        def rejoins(tok, d):
            if match_position(tokens[1:m + 1], 1, tok, d) is not None:
                return True
            return any(match_position(bt, d0, tok, d) is not None for d0, bt in grown)

        for j, second in marks:
            if len(tokens) >= n_nodes:
                break
            tokens.append(second)
            parent.append(j - 1)
            depth.append(j)
            btoks = [second]
            while not rejoins(btoks[-1], j + len(btoks) - 1) and len(btoks) < max_branch and len(tokens) < n_nodes:
                ids, _ = self.tree_top2(tokens, parent)        # the whole tree; the branch tip is its last node
                tokens.append(int(ids[-1, 0]))
                parent.append(len(tokens) - 2)
                depth.append(j + len(btoks))
                btoks.append(int(ids[-1, 0]))
            grown.append((j, btoks))
        return {"tokens": np.asarray(tokens, np.int32), "parent": np.asarray(parent, np.int32),
                "depth": np.asarray(depth, np.int64), "marks": marks, "trunk_len": m}

    def recycled_draft(self, last_accepted, seq1, accept_len, bonus, max_len, max_regen):
        """Section IV-B: the unaccepted tail of the old draft (sequence 1, which keeps being extended) and the
        regeneration from the target's token (sequence 2) are decoded side by side as two chains of one masked token
        tree under the last accepted token; when a regenerated token equals sequence 1's token at the same or an
        adjacent depth the sequences are merged and the rest of sequence 1 is reused."""
        seq1 = [int(t) for t in seq1]
        a = int(accept_len)
        tail = seq1[a:]
        if not tail:
            return {"draft": [], "steps": 0, "merged_at": None, "regenerated": [], "extended": []}
        regen, ext = [], []
        merged = None
        for _ in range(max_regen):
            c1 = tail + ext
            c2 = [int(bonus)] + regen
            tokens = [int(last_accepted)] + c1 + c2
            parent = [-1] + [0] + list(range(1, len(c1))) + [0] + list(range(len(c1) + 1, len(c1) + len(c2)))
            ids, _ = self.tree_top2(tokens, parent)
            ext.append(int(ids[len(c1), 0]))
            r = int(ids[len(c1) + len(c2), 0])
            regen.append(r)
            q = a + 1 + len(regen)
            hit = match_position(tail + ext, a + 1, r, q, lowest_pos=a + 1)
            if hit is not None:
                merged = a + 1 + hit
                break
            if len(regen) >= max_len:
                break
        draft = regen + (tail + ext)[merged - a:] if merged is not None else list(regen)
        return {"draft": draft[:max_len], "steps": len(regen), "merged_at": merged, "regenerated": regen, "extended": ext}
