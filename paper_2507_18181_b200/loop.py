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

    def run_draft(self, feeds):
        """feeds: {b: tokens} -- tokens the draft model of utterance b consumes this round, one per autoregressive step.
        Step j runs every utterance that still has a token left as one batched call of single-node trees and
        appends that token's K/V to its draft cache.  (The proposer supplies the draft tokens, so the draft
        model's own arg-max is not read back.)"""
        if self.draft_kvs is None:
            return
        steps = max((len(f) for f in feeds.values()), default=0)
        for j in range(steps):
            members = [b for b in sorted(feeds) if len(feeds[b]) > j]
            bv = self._verifier(self.draft_kvs, members)
            toks = torch.tensor([int(feeds[b][j]) for b in members], dtype=torch.int32, device=self.device)
            bv.verify(toks, self._minus_one[:len(members)], list(range(len(members) + 1)))
            bv.commit()
            for b in members:
                self.draft_len[b] += 1
                self.draft_dev_len[b] += 1
            self.draft_steps += 1

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
            trees, feeds = {}, {}
            for b in active:
                tokens, parent, feed = proposer.propose(b, emitted[b])
                assert int(tokens[0]) == history[b][-1]
                trees[b] = (tokens, parent)
                feeds[b] = feed
                self.align_draft(b, history[b])
            self.run_draft(feeds)
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
        vocab = self.draft_kvs[0].model.cfg.vocab
        trunk = {b: [] for b in members}
        branch = {b: None for b in members}            # (depth of the parent on the trunk, token)
        cur = {b: int(roots[b]) for b in members}
        live = list(members)
        for _ in range(max_len):
            if not live:
                break
            bv = self._verifier(self.draft_kvs, live)
            nb = len(live)
            if not hasattr(bv, "logits"):
                bv.logits = torch.empty(nb, vocab, dtype=torch.float32, device=self.device)
                bv.top_ids = torch.empty(nb, 2, dtype=torch.int32, device=self.device)
                bv.top_probs = torch.empty(nb, 2, dtype=torch.float32, device=self.device)
            toks = torch.tensor([cur[b] for b in live], dtype=torch.int32, device=self.device)
            bv.verify(toks, self._minus_one[:nb], list(range(nb + 1)), bv.logits)
            bv.commit()
            B.specasr_top2_probs(bv.logits.data_ptr(), nb, vocab, bv.top_ids.data_ptr(), bv.top_probs.data_ptr(),
                                 DeviceKV._stream())
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
