"""ctypes wrapper around the C oracle (`ps_oracle.c`).  Test infrastructure only.

Argument marshalling only: every step is computed by the C file.  Arrays are
numpy (or CPU torch tensors, converted without copying where the dtype matches).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ps_oracle.c")
_LIB = os.path.join(_HERE, "libps_oracle.so")
_lib = None

STATUS = {0: "ok", 1: "invalid argument", 2: "key out of range", 3: "worker out of range",
          4: "partition full"}


def build_oracle(force: bool = False) -> str:
    """Compile the oracle with gcc (plain C99, -O2, no fast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-std=c99", "-O2", "-fPIC", "-shared", "-Wall", "-Wextra",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = C.CDLL(build_oracle())
        vp, u64, u32, f32 = C.c_void_p, C.c_uint64, C.c_uint32, C.c_float
        lib.ops_create.restype = vp
        lib.ops_create.argtypes = [u64, u32, u32, u64]
        lib.ops_destroy.argtypes = [vp]
        lib.ops_init_range_partition.argtypes = [vp]
        for name, args in {
            "ops_set_rows": [vp, vp, u64, vp],
            "ops_pull": [vp, vp, u64, vp],
            "ops_push": [vp, vp, u64, vp],
            "ops_localize": [vp, u32, vp, u64],
            "ops_get_location": [vp, vp, u64, vp, vp],
            "ops_step_mf": [vp, vp, vp, vp, u64, u64, f32, f32, vp],
            "ops_step_kge": [vp, vp, vp, vp, vp, vp, u64, u32, u64, u32, f32, f32, vp],
            "ops_step_rescal": [vp, vp, vp, vp, vp, vp, u64, u32, u64, u32, f32, f32, vp],
            "ops_step_sgns": [vp, vp, u64, u64, u64, u32, vp, u32, u64, f32, vp],
        }.items():
            getattr(lib, name).argtypes = args
            getattr(lib, name).restype = C.c_int
        for name in ("ops_rows", "ops_owner", "ops_slot", "ops_stack", "ops_top"):
            getattr(lib, name).argtypes = [vp]
            getattr(lib, name).restype = vp
        _lib = lib
    return _lib


def _np(a, dtype):
    """Contiguous numpy array of `dtype` viewing (or converting) `a`."""
    if hasattr(a, "detach"):                     # torch tensor on the CPU
        a = a.detach().cpu().numpy()
    a = np.asarray(a)
    if a.dtype != dtype:
        if a.dtype.itemsize == np.dtype(dtype).itemsize and a.dtype.kind in "iu" and np.dtype(dtype).kind in "iu":
            a = a.view(dtype)                    # int32 <-> uint32, int64 <-> uint64
        else:
            a = a.astype(dtype)
    return np.ascontiguousarray(a)


def _p(a):
    return a.ctypes.data_as(C.c_void_p)


class OracleError(RuntimeError):
    def __init__(self, code):
        super().__init__(f"oracle: {STATUS.get(code, code)}")
        self.code = code


class OracleStore:
    """The oracle's parameter store: rows by key, location table, free-slot stacks."""

    def __init__(self, num_keys: int, row_len: int, num_workers: int = 1, slots_per_part: int | None = None):
        lib = _load()
        part = (num_keys + num_workers - 1) // num_workers
        self.K, self.L, self.N = num_keys, row_len, num_workers
        self.S = part if slots_per_part is None else slots_per_part
        self._h = lib.ops_create(self.K, self.L, self.N, self.S)
        if not self._h:
            raise ValueError("oracle: bad store configuration")
        lib.ops_init_range_partition(self._h)
        self.loss = np.zeros(1, dtype=np.float64)

    def close(self):
        if self._h:
            _load().ops_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @staticmethod
    def _check(code):
        if code != 0:
            raise OracleError(code)

    # raw views (no copy) -----------------------------------------------------
    def _view(self, fn, ctype, shape):
        ptr = C.cast(getattr(_load(), fn)(self._h), C.POINTER(ctype))
        return np.ctypeslib.as_array(ptr, shape=shape)

    @property
    def rows(self):
        return self._view("ops_rows", C.c_float, (self.K, self.L))

    @property
    def owner(self):
        return self._view("ops_owner", C.c_uint32, (self.K,))

    @property
    def slot(self):
        return self._view("ops_slot", C.c_uint32, (self.K,))

    @property
    def stack(self):
        return self._view("ops_stack", C.c_uint32, (self.N, self.S))

    @property
    def top(self):
        return self._view("ops_top", C.c_uint64, (self.N,))

    # primitives --------------------------------------------------------------
    def set_rows(self, keys, vals):
        keys, vals = _np(keys, np.uint64), _np(vals, np.float32)
        assert vals.size == keys.size * self.L
        self._check(_load().ops_set_rows(self._h, _p(keys), keys.size, _p(vals)))

    def pull(self, keys):
        keys = _np(keys, np.uint64)
        out = np.empty((keys.size, self.L), dtype=np.float32)
        self._check(_load().ops_pull(self._h, _p(keys), keys.size, _p(out)))
        return out

    def push(self, keys, updates):
        keys, updates = _np(keys, np.uint64), _np(updates, np.float32)
        assert updates.size == keys.size * self.L
        self._check(_load().ops_push(self._h, _p(keys), keys.size, _p(updates)))

    def localize(self, worker, keys):
        keys = _np(keys, np.uint64)
        self._check(_load().ops_localize(self._h, int(worker), _p(keys), keys.size))

    def get_location(self, keys):
        keys = _np(keys, np.uint64)
        owner = np.empty(keys.size, dtype=np.uint32)
        slot = np.empty(keys.size, dtype=np.uint32)
        self._check(_load().ops_get_location(self._h, _p(keys), keys.size, _p(owner), _p(slot)))
        return owner, slot

    # training steps ----------------------------------------------------------
    def step_mf(self, i, j, v, col_key_base, lr, lam):
        i, j, v = _np(i, np.uint32), _np(j, np.uint32), _np(v, np.float32)
        self._check(_load().ops_step_mf(self._h, _p(i), _p(j), _p(v), i.size, int(col_key_base),
                                        float(lr), float(lam), _p(self.loss)))

    def step_kge(self, s, r, o, neg_ent, neg_side, rel_key_base, dim, lr, eps):
        s, r, o = _np(s, np.uint32), _np(r, np.uint32), _np(o, np.uint32)
        neg_ent, neg_side = _np(neg_ent, np.uint32), _np(neg_side, np.uint8)
        n_neg = neg_ent.size // max(s.size, 1)
        assert neg_ent.size == s.size * n_neg == neg_side.size
        self._check(_load().ops_step_kge(self._h, _p(s), _p(r), _p(o), _p(neg_ent), _p(neg_side), s.size,
                                         n_neg, int(rel_key_base), int(dim), float(lr), float(eps),
                                         _p(self.loss)))

    def step_rescal(self, s, r, o, neg_ent, neg_side, rel_key_base, dim, lr, eps):
        s, r, o = _np(s, np.uint32), _np(r, np.uint32), _np(o, np.uint32)
        neg_ent, neg_side = _np(neg_ent, np.uint32), _np(neg_side, np.uint8)
        n_neg = neg_ent.size // max(s.size, 1)
        assert neg_ent.size == s.size * n_neg == neg_side.size
        self._check(_load().ops_step_rescal(self._h, _p(s), _p(r), _p(o), _p(neg_ent), _p(neg_side), s.size,
                                            n_neg, int(rel_key_base), int(dim), float(lr), float(eps),
                                            _p(self.loss)))

    def step_sgns(self, tokens, first_pos, n_centers, window, negs, n_neg, out_key_base, lr):
        tokens, negs = _np(tokens, np.uint32), _np(negs, np.uint32)
        self._check(_load().ops_step_sgns(self._h, _p(tokens), int(first_pos), int(n_centers), tokens.size,
                                          int(window), _p(negs), int(n_neg), int(out_key_base), float(lr),
                                          _p(self.loss)))
