"""CPU oracle of the sparse-map front end of the store.  Test infrastructure only.

The paper's servers keep their local parameters "in dense arrays or sparse maps"
(Section 3.7): dense arrays when keys are contiguous, a map when they are not.
Here the map is a translation of arbitrary 64-bit keys to the dense keys of the
store: a key gets the next unused dense key the first time it is seen, so dense
keys are handed out in order of first appearance (the paper prescribes no order;
this reading is fixed for this repository and stated as such: parity unpinned
by the paper, pinned by the definition below and by brute force).

Plain Python on purpose: a dict and a list, one key at a time.
"""
from __future__ import annotations

import numpy as np

ABSENT = np.uint64(0xFFFFFFFFFFFFFFFF)


class KeyMapFull(Exception):
    pass


class OracleKeyMap:
    def __init__(self, capacity: int):
        self.capacity = int(capacity)
        self.dense_of: dict[int, int] = {}
        self.sparse_of: list[int] = []          # dense key -> sparse key

    def __len__(self):
        return len(self.sparse_of)

    def insert(self, keys) -> np.ndarray:
        """Dense key of every occurrence; unseen keys are added in order of first occurrence.  A call that would
        exceed the capacity raises KeyMapFull and adds nothing."""
        keys = [int(k) for k in np.asarray(keys, dtype=np.uint64).ravel()]
        fresh = []
        seen = set()
        for k in keys:
            if k not in self.dense_of and k not in seen:
                seen.add(k)
                fresh.append(k)
        if len(self.sparse_of) + len(fresh) > self.capacity:
            raise KeyMapFull(f"{len(self.sparse_of)} + {len(fresh)} keys > capacity {self.capacity}")
        for k in fresh:
            self.dense_of[k] = len(self.sparse_of)
            self.sparse_of.append(k)
        return np.array([self.dense_of[k] for k in keys], dtype=np.uint64)

    def lookup(self, keys) -> np.ndarray:
        """Dense key of every occurrence, ABSENT for keys never inserted."""
        keys = np.asarray(keys, dtype=np.uint64).ravel()
        return np.array([self.dense_of.get(int(k), int(ABSENT)) for k in keys], dtype=np.uint64)
