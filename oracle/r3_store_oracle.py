"""CPU oracle for the routing-record store of Section 4.2 (router-mask caching with the prefix
KV cache, multi-turn reuse).

TEST INFRASTRUCTURE ONLY (same rules as r3_oracle.py).  Pure Python / numpy, written for
obviousness: a store is a dict from page number to a [L, page_tokens, K] array; a sequence is a
list of page numbers; prefix sharing is two sequences listing the same page numbers.

What Section 4.2 fixes: "for each layer and token prefix, the corresponding routing masks are
stored with KVCache; when the same prefix occurs and hits the cache, the masks can be reused".
What it leaves open and is read here as in paged KV caches: records live in fixed-size pages of
`page_tokens` tokens (all layers of a token together in its page), a prefix is shared in whole
pages, a page is identified by the token ids of everything up to its end, and a page returns to
the free list when the last sequence using it is closed.
"""
from __future__ import annotations

import numpy as np


def append(pages: dict, table: list, n_have: int, rec_new: np.ndarray, page_tokens: int) -> int:
    """Writes rec_new [L, n_new, K] as tokens n_have .. n_have+n_new-1 of the sequence whose page
    numbers are `table` (long enough).  Returns the new length."""
    L, n_new, K = rec_new.shape
    for i in range(n_new):
        pos = n_have + i
        page = pages[table[pos // page_tokens]]
        for l in range(L):
            page[l, pos % page_tokens, :] = rec_new[l, i, :]
    return n_have + n_new


def gather(pages: dict, tables: list, lengths: list, page_tokens: int, L: int, K: int, dtype):
    """The packed training batch [L, sum(lengths), K]: sequence after sequence, token after token."""
    out = np.zeros((L, int(sum(lengths)), K), dtype=dtype)
    at = 0
    for table, n in zip(tables, lengths):
        for pos in range(n):
            page = pages[table[pos // page_tokens]]
            out[:, at, :] = page[:, pos % page_tokens, :]
            at += 1
    return out


class PrefixIndex:
    """Which page holds the records of a given token prefix.  A page is keyed by the tuple of ALL
    token ids up to and including its own (so equal keys mean equal prefixes)."""

    def __init__(self, n_pages: int, page_tokens: int):
        self.page_tokens = page_tokens
        self.free = list(range(n_pages))
        self.ref = {}
        self.by_prefix = {}
        self.key_of = {}

    def match(self, token_ids) -> list:
        """Pages of the longest cached whole-page prefix of token_ids (their use count goes up)."""
        got = []
        for end in range(self.page_tokens, len(token_ids) + 1, self.page_tokens):
            page = self.by_prefix.get(tuple(token_ids[:end]))
            if page is None:
                break
            got.append(page)
        for p in got:
            self.ref[p] += 1
        return got

    def alloc(self, n: int) -> list:
        if n > len(self.free):
            raise MemoryError("out of pages")
        out = [self.free.pop(0) for _ in range(n)]
        for p in out:
            self.ref[p] = 1
        return out

    def publish(self, token_ids, table) -> None:
        """Registers every full page of the sequence so that later sequences can share it."""
        for i, page in enumerate(table):
            end = (i + 1) * self.page_tokens
            if end > len(token_ids):
                break
            key = tuple(token_ids[:end])
            if key not in self.by_prefix and page not in self.key_of:
                self.by_prefix[key] = page
                self.key_of[page] = key

    def release(self, table) -> None:
        for p in table:
            self.ref[p] -= 1
            if self.ref[p] == 0:
                del self.ref[p]
                key = self.key_of.pop(p, None)
                if key is not None:
                    del self.by_prefix[key]
                self.free.append(p)
