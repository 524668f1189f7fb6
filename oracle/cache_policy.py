"""CPU oracle of the online n-gram cache: insertion of unseen n-grams (Algorithm 1,
cache-update line) and bounded size with LRU / LFU eviction (App. D.5, cache
scalability).

TEST INFRASTRUCTURE ONLY: a Python dictionary with the policy written out, shared
with nothing on the CUDA side.

What the paper fixes: an n-gram (t, [d_1..d_n]) is added when it is not in the cache
yet; LRU evicts the n-gram that has not been accessed for the longest time, LFU the
one with the lowest access frequency; the cache has a maximum size.

Readings where it is silent:
  * an ACCESS is a lookup hit that the translation actually uses (a cached run that
    the merge scan of Eq. (1) merges), and the insertion itself; probes that hit but
    lose to a longer run do not count;
  * time is a clock the caller advances (one tick per verification step); an access
    stamps the entry with the current clock; the frequency starts at 1 on insertion
    and grows by 1 per access;
  * eviction happens in an explicit trim: with size - max_entries = k > 0, the k
    entries that come first in the order (inserted at the current clock?, score, run
    key) are removed, where score = last-access clock (LRU) or frequency (LFU).
    Entries inserted at the current clock come last, so a trim never throws out what
    the same step has just learnt unless nothing else is left; equal scores are
    broken by the run's packed key (id + 1 in 16 bits per position, first id lowest),
    an arbitrary but total order;
  * within one batch of insertions the first candidate with a given run wins; a
    candidate with a malformed run (length outside 2..4, id outside the vocabulary)
    is skipped.

Pins (tests/test_oracle_cache_policy.py): trim after every insertion of one item
reproduces a textbook LRU (collections.OrderedDict) and a brute-force LFU; the trim
keeps exactly max_entries entries and never evicts a strictly better entry while
keeping a worse one; first-wins; the tracked translation equals the static one.
"""
from __future__ import annotations

from typing import Dict, Iterable, List, Optional, Sequence, Tuple

LRU, LFU = 0, 1
N_MAX = 4


def packed_key(run: Sequence[int]) -> int:
    k = 0
    for j, d in enumerate(run):
        k |= (int(d) + 1) << (16 * j)
    return k


class DynamicCache:
    def __init__(self, max_entries: int, policy: int, draft_vocab: int, target_vocab: int):
        assert policy in (LRU, LFU)
        self.max_entries, self.policy = int(max_entries), policy
        self.v_q, self.v_p = draft_vocab, target_vocab
        self.clock = 0
        # run (tuple of draft ids) -> [target, last-access clock, frequency, clock of insertion]
        self.entries: Dict[Tuple[int, ...], List[int]] = {}

    def __len__(self):
        return len(self.entries)

    def set_clock(self, clock: int):
        self.clock = int(clock)

    def lookup(self, run: Sequence[int]) -> int:
        e = self.entries.get(tuple(int(x) for x in run))
        return -1 if e is None else e[0]

    def touch(self, run: Sequence[int]):
        e = self.entries[tuple(int(x) for x in run)]
        e[1] = max(e[1], self.clock)
        e[2] += 1

    def insert_batch(self, runs, lengths, targets) -> int:
        """Candidates in order; returns how many were new."""
        added = 0
        for run, n, t in zip(runs, lengths, targets):
            n = int(n)
            if n < 2 or n > N_MAX:
                continue
            key = tuple(int(x) for x in run[:n])
            if any(d < 0 or d >= self.v_q for d in key) or not (0 <= int(t) < self.v_p):
                continue
            if key in self.entries:
                continue                                    # only unseen n-grams are added
            self.entries[key] = [int(t), self.clock, 1, self.clock]
            added += 1
        return added

    def _order(self, item):
        key, (target, stamp, freq, born) = item
        score = stamp if self.policy == LRU else freq
        return (1 if born == self.clock else 0, score, packed_key(key))

    def trim(self) -> int:
        k = len(self.entries) - self.max_entries
        if k <= 0:
            return 0
        victims = sorted(self.entries.items(), key=self._order)[:k]
        for key, _ in victims:
            del self.entries[key]
        return k

    def map_sequence(self, vocab_map, draft_ids, q_sel):
        """Eq. (1) with this cache (greedy, longest cached run first, cache before the
        direct map), stamping the runs it merges.  Returns (tgt, q_prime, span_start,
        span_len, m, unmapped_stop)."""
        d = [int(x) for x in draft_ids]
        K = len(d)
        tgt, qp, ss, sl = [], [], [], []
        s = 0
        stop = False
        while s < K:
            hit = 0
            for L in range(N_MAX, 1, -1):
                if s + L > K or any(x < 0 or x >= self.v_q for x in d[s:s + L]):
                    continue
                t = self.lookup(d[s:s + L])
                if t >= 0:
                    self.touch(d[s:s + L])
                    prod = 1.0
                    for j in range(L):
                        prod *= float(q_sel[s + j])
                    tgt.append(t); qp.append(prod); ss.append(s); sl.append(L)
                    s += L
                    hit = L
                    break
            if hit:
                continue
            direct = int(vocab_map[d[s]]) if 0 <= d[s] < self.v_q else -1
            if direct >= 0:
                tgt.append(direct); qp.append(float(q_sel[s])); ss.append(s); sl.append(1)
                s += 1
            else:
                ss.append(s); stop = True
                break
        return tgt, qp, ss, sl, len(tgt), stop
