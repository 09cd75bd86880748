"""Python binding of the C interface in include/ps.h: argument marshalling only.

Every function here has the name and the argument order of the C entry point it
calls; tensors are passed as raw device (or host) pointers, the stream as the
current torch CUDA stream.  Nothing is computed in Python.  There is no
fallback: if the CUDA library has not been built, loading it raises.

`Store` is a small convenience wrapper that lets torch own the four device
buffers a store needs (torch is used for device memory and streams only).
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libps_b200.so")

PS_OK = 0
PS_ERR_INVALID_ARG = 1
PS_ERR_KEY_RANGE = 2
PS_ERR_WORKER_RANGE = 3
PS_ERR_CAPACITY = 4
PS_ERR_WORKSPACE = 5
PS_ERR_CUDA = 6
PS_ERR_UNSUPPORTED = 7
PS_MF_AUTO, PS_MF_BY_COLUMN, PS_MF_SYMMETRIC, PS_MF_SYMMETRIC_ROW_COPIES = 0, 1, 2, 3
PS_PUSH_SORTED, PS_PUSH_ATOMIC = 0, 1
PS_PUSH_STATIC_MAX_KEYS = 16384
PS_PUSH_STATIC_MAX_ROW_LEN = 256


class ps_config_t(C.Structure):
    _fields_ = [("num_keys", C.c_uint64), ("row_len", C.c_uint32), ("num_workers", C.c_uint32),
                ("slots_per_part", C.c_uint64), ("device", C.c_int32)]


class ps_sizes_t(C.Structure):
    _fields_ = [("store_bytes", C.c_size_t), ("table_bytes", C.c_size_t), ("freelist_bytes", C.c_size_t),
                ("workspace_bytes", C.c_size_t)]


_vp, _u64, _u32, _f32, _sz = C.c_void_p, C.c_uint64, C.c_uint32, C.c_float, C.c_size_t

# name -> (restype, argtypes); mirrors include/ps.h declaration by declaration
SIGNATURES = {
    "ps_query_sizes": (C.c_int, [C.POINTER(ps_config_t), _u64, C.POINTER(ps_sizes_t)]),
    "ps_create": (C.c_int, [C.POINTER(ps_config_t), _vp, _vp, _vp, _vp, _sz, _u64, C.POINTER(_vp)]),
    "ps_destroy": (C.c_int, [_vp]),
    "ps_init_range_partition": (C.c_int, [_vp, _vp]),
    "ps_set_rows": (C.c_int, [_vp, _vp, _u64, _vp, _vp]),
    "ps_pull": (C.c_int, [_vp, _vp, _u64, _vp, _vp]),
    "ps_push": (C.c_int, [_vp, _vp, _u64, _vp, _vp]),
    "ps_localize": (C.c_int, [_vp, _u32, _vp, _u64, _vp]),
    "ps_localize_beside": (C.c_int, [_vp, _u32, _vp, _u64, _vp]),
    "ps_localize_stats": (C.c_int, [_vp, _vp]),
    "ps_step_mf": (C.c_int, [_vp, _vp, _vp, _vp, _u64, _u64, _f32, _f32, _vp, _vp]),
    "ps_step_kge": (C.c_int, [_vp, _vp, _vp, _vp, _vp, _vp, _u64, _u32, _u64, _u32, _f32, _f32, _vp, _vp]),
    "ps_step_rescal": (C.c_int, [_vp, _vp, _vp, _vp, _vp, _vp, _u64, _u32, _u64, _u32, _f32, _f32, _vp, _vp]),
    "ps_step_sgns": (C.c_int, [_vp, _vp, _u64, _u64, _u64, _u32, _vp, _u32, _u64, _f32, _vp, _vp]),
    "ps_step_mf_host": (C.c_int, [_vp, _vp, _vp, _vp, _u64, _u64, _f32, _f32, _vp, _vp, _vp]),
    "ps_step_kge_host": (C.c_int, [_vp, _vp, _vp, _vp, _vp, _vp, _u64, _u32, _u64, _u32, _f32, _f32, _vp, _vp, _vp]),
    "ps_step_sgns_host": (C.c_int, [_vp, _vp, _u64, _u64, _u64, _u64, _u64, _u32, _vp, _u64, _u32, _u64, _f32, _vp,
                                    _vp, _vp]),
    "ps_push_static": (C.c_int, [_vp, _vp, _u64, _u32, _u64, _vp, _u64, _vp, _vp]),
    "ps_get_location": (C.c_int, [_vp, _vp, _u64, _vp, _vp, _vp]),
    "ps_export": (C.c_int, [_vp, _vp, _vp, _vp]),
    "ps_export_freelists": (C.c_int, [_vp, _vp, _vp]),
    "ps_sync": (C.c_int, [_vp, _vp]),
    "ps_set_pipelining": (C.c_int, [_vp, C.c_int]),
    "ps_set_host_overlap": (C.c_int, [_vp, C.c_int]),
    "ps_set_mf_path": (C.c_int, [_vp, C.c_int]),
    "ps_set_push_mode": (C.c_int, [_vp, C.c_int]),
    "ps_selftest_barrier_timeout": (C.c_int, [_vp, _vp]),
    "ps_launch_count": (C.c_uint64, [_vp]),
    "ps_rows_moved": (C.c_int, [_vp, C.POINTER(_u64)]),
    "ps_profile_start": (C.c_int, [_vp, _u32]),
    "ps_profile_stop": (C.c_int, [_vp, C.c_char_p, _sz]),
    "ps_dsgd_epoch_mf": (C.c_int, [_vp, _vp, _vp, _vp, _vp, _u64, _u64, _u64, _f32, _f32, _vp, _vp]),
    "ps_keymap_query_bytes": (C.c_int, [_u64, _u64, C.POINTER(_sz)]),
    "ps_keymap_create": (C.c_int, [_u64, _u64, _vp, _sz, C.c_int32, _vp, C.POINTER(_vp)]),
    "ps_keymap_destroy": (C.c_int, [_vp]),
    "ps_keymap_insert": (C.c_int, [_vp, _vp, _u64, _vp, _vp]),
    "ps_keymap_lookup": (C.c_int, [_vp, _vp, _u64, _vp, _vp]),
    "ps_keymap_sync": (C.c_int, [_vp, _vp, C.POINTER(_u64)]),
    "ps_keymap_launch_count": (C.c_uint64, [_vp]),
    "ps_status_string": (C.c_char_p, [C.c_int]),
}

_lib = None


def load_library() -> C.CDLL:
    """Loads libps_b200.so; raises if it has not been built (there is no other code path)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2002_00655_b200.build`")
        lib = C.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype, fn.argtypes = res, args
        _lib = lib
    return _lib


class PSError(RuntimeError):
    def __init__(self, code: int, where: str):
        msg = load_library().ps_status_string(code).decode()
        super().__init__(f"{where}: {msg} (status {code})")
        self.code = code


def _check(code: int, where: str) -> None:
    if code != PS_OK:
        raise PSError(code, where)


def _dptr(t, dtype=None):
    """Device pointer of a contiguous CUDA tensor (None -> NULL)."""
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "expected a contiguous CUDA tensor"
    if dtype is not None:
        assert t.dtype in dtype, f"expected dtype in {dtype}, got {t.dtype}"
    return t.data_ptr()


def _hptr(t, dtype=None):
    """Host pointer of a contiguous CPU tensor (None -> NULL)."""
    if t is None:
        return None
    assert (not t.is_cuda) and t.is_contiguous(), "expected a contiguous CPU tensor"
    if dtype is not None:
        assert t.dtype in dtype, f"expected dtype in {dtype}, got {t.dtype}"
    return t.data_ptr()


def _stream():
    return torch.cuda.current_stream().cuda_stream


_U32 = (torch.int32, torch.uint32)
_U64 = (torch.int64, torch.uint64)
_F32 = (torch.float32,)
_F64 = (torch.float64,)
_U8 = (torch.uint8,)


# ---- one function per C entry point -------------------------------------------------
def ps_query_sizes(cfg: ps_config_t, max_batch_keys: int) -> ps_sizes_t:
    out = ps_sizes_t()
    _check(load_library().ps_query_sizes(C.byref(cfg), max_batch_keys, C.byref(out)), "ps_query_sizes")
    return out


def ps_create(cfg, d_store, d_table, d_freelists, d_workspace, max_batch_keys):
    h = _vp()
    _check(load_library().ps_create(C.byref(cfg), _dptr(d_store), _dptr(d_table), _dptr(d_freelists),
                                    _dptr(d_workspace), d_workspace.numel() * d_workspace.element_size(),
                                    max_batch_keys, C.byref(h)), "ps_create")
    return h


def ps_destroy(ps):
    _check(load_library().ps_destroy(ps), "ps_destroy")


def ps_init_range_partition(ps):
    _check(load_library().ps_init_range_partition(ps, _stream()), "ps_init_range_partition")


def ps_set_rows(ps, d_keys, d_vals):
    _check(load_library().ps_set_rows(ps, _dptr(d_keys, _U64), d_keys.numel(), _dptr(d_vals, _F32), _stream()),
           "ps_set_rows")


def ps_pull(ps, d_keys, d_out):
    _check(load_library().ps_pull(ps, _dptr(d_keys, _U64), d_keys.numel(), _dptr(d_out, _F32), _stream()), "ps_pull")


def ps_push(ps, d_keys, d_updates):
    _check(load_library().ps_push(ps, _dptr(d_keys, _U64), d_keys.numel(), _dptr(d_updates, _F32), _stream()),
           "ps_push")


def ps_localize(ps, worker, d_keys):
    _check(load_library().ps_localize(ps, worker, _dptr(d_keys, _U64), d_keys.numel(), _stream()), "ps_localize")


def ps_localize_beside(ps, worker, d_keys, loc_stream):
    """loc_stream: a torch.cuda.Stream other than the current one."""
    _check(load_library().ps_localize_beside(ps, worker, _dptr(d_keys, _U64), d_keys.numel(), loc_stream.cuda_stream),
           "ps_localize_beside")


class ps_localize_stats_t(C.Structure):
    _fields_ = [(n, C.c_uint64) for n in ("requested", "moved", "already_local", "moved_again", "deferred")]


def ps_localize_stats(ps) -> dict:
    out = ps_localize_stats_t()
    _check(load_library().ps_localize_stats(ps, C.byref(out)), "ps_localize_stats")
    return {n: getattr(out, n) for n, _ in out._fields_}


def ps_step_mf(ps, d_i, d_j, d_v, col_key_base, lr, lam, d_loss_accum=None):
    _check(load_library().ps_step_mf(ps, _dptr(d_i, _U32), _dptr(d_j, _U32), _dptr(d_v, _F32), d_i.numel(),
                                     col_key_base, lr, lam, _dptr(d_loss_accum, _F64), _stream()), "ps_step_mf")


def ps_step_kge(ps, d_s, d_r, d_o, d_neg_ent, d_neg_side, n_neg, rel_key_base, dim_complex, lr, eps,
                d_loss_accum=None):
    _check(load_library().ps_step_kge(ps, _dptr(d_s, _U32), _dptr(d_r, _U32), _dptr(d_o, _U32),
                                      _dptr(d_neg_ent, _U32), _dptr(d_neg_side, _U8), d_s.numel(), n_neg,
                                      rel_key_base, dim_complex, lr, eps, _dptr(d_loss_accum, _F64), _stream()),
           "ps_step_kge")


def ps_step_rescal(ps, d_s, d_r, d_o, d_neg_ent, d_neg_side, n_neg, rel_key_base, dim, lr, eps, d_loss_accum=None):
    _check(load_library().ps_step_rescal(ps, _dptr(d_s, _U32), _dptr(d_r, _U32), _dptr(d_o, _U32),
                                         _dptr(d_neg_ent, _U32), _dptr(d_neg_side, _U8), d_s.numel(), n_neg,
                                         rel_key_base, dim, lr, eps, _dptr(d_loss_accum, _F64), _stream()),
           "ps_step_rescal")


def ps_step_sgns(ps, d_tokens, first_pos, n_centers, window, d_negs, n_neg, out_key_base, lr, d_loss_accum=None):
    _check(load_library().ps_step_sgns(ps, _dptr(d_tokens, _U32), first_pos, n_centers, d_tokens.numel(), window,
                                       _dptr(d_negs, _U32), n_neg, out_key_base, lr, _dptr(d_loss_accum, _F64),
                                       _stream()), "ps_step_sgns")


def ps_step_mf_host(ps, h_i, h_j, h_v, col_key_base, lr, lam, d_loss_accum, h_loss):
    _check(load_library().ps_step_mf_host(ps, _hptr(h_i, _U32), _hptr(h_j, _U32), _hptr(h_v, _F32), h_i.numel(),
                                          col_key_base, lr, lam, _dptr(d_loss_accum, _F64), _hptr(h_loss, _F64),
                                          _stream()), "ps_step_mf_host")


def ps_step_kge_host(ps, h_s, h_r, h_o, h_neg_ent, h_neg_side, n_neg, rel_key_base, dim_complex, lr, eps,
                     d_loss_accum, h_loss):
    _check(load_library().ps_step_kge_host(ps, _hptr(h_s, _U32), _hptr(h_r, _U32), _hptr(h_o, _U32),
                                           _hptr(h_neg_ent, _U32), _hptr(h_neg_side, _U8), h_s.numel(), n_neg,
                                           rel_key_base, dim_complex, lr, eps, _dptr(d_loss_accum, _F64),
                                           _hptr(h_loss, _F64), _stream()), "ps_step_kge_host")


def ps_step_sgns_host(ps, h_tokens, tok_first, first_pos, n_centers, corpus_len, window, h_negs, n_neg,
                      out_key_base, lr, d_loss_accum, h_loss):
    _check(load_library().ps_step_sgns_host(ps, _hptr(h_tokens, _U32), tok_first, h_tokens.numel(), first_pos,
                                            n_centers, corpus_len, window, _hptr(h_negs, _U32), h_negs.numel(),
                                            n_neg, out_key_base, lr, _dptr(d_loss_accum, _F64),
                                            _hptr(h_loss, _F64), _stream()), "ps_step_sgns_host")


def ps_push_static(d_store, d_table, num_keys, row_len, slots_per_part, d_keys, d_updates) -> int:
    """Handle-free push that allocates nothing (static scratch inside the library); returns the status code."""
    return load_library().ps_push_static(_dptr(d_store, _F32), _dptr(d_table), num_keys, row_len, slots_per_part,
                                         _dptr(d_keys, _U64), d_keys.numel(), _dptr(d_updates, _F32), _stream())


def ps_get_location(ps, d_keys, d_owner, d_slot):
    _check(load_library().ps_get_location(ps, _dptr(d_keys, _U64), d_keys.numel(), _dptr(d_owner, _U32),
                                          _dptr(d_slot, _U32), _stream()), "ps_get_location")


def ps_export(ps, h_rows_by_key=None, h_owner=None, h_slot=None):
    _check(load_library().ps_export(ps, _hptr(h_rows_by_key, _F32), _hptr(h_owner, _U32), _hptr(h_slot, _U32)),
           "ps_export")


def ps_export_freelists(ps, h_stacks=None, h_tops=None):
    _check(load_library().ps_export_freelists(ps, _hptr(h_stacks, _U32), _hptr(h_tops, _U64)),
           "ps_export_freelists")


def ps_sync(ps) -> int:
    """Waits for the current stream; returns (and clears) the first error latched on the device."""
    return load_library().ps_sync(ps, _stream())


def ps_set_host_overlap(ps, on: bool) -> None:
    _check(load_library().ps_set_host_overlap(ps, 1 if on else 0), "ps_set_host_overlap")


def ps_set_pipelining(ps, on: bool) -> None:
    _check(load_library().ps_set_pipelining(ps, 1 if on else 0), "ps_set_pipelining")


def ps_set_push_mode(ps, mode: int) -> None:
    _check(load_library().ps_set_push_mode(ps, int(mode)), "ps_set_push_mode")


def ps_set_mf_path(ps, path: int) -> None:
    _check(load_library().ps_set_mf_path(ps, int(path)), "ps_set_mf_path")


def ps_selftest_barrier_timeout(ps) -> None:
    _check(load_library().ps_selftest_barrier_timeout(ps, _stream()), "ps_selftest_barrier_timeout")


def ps_launch_count(ps) -> int:
    return load_library().ps_launch_count(ps)


def ps_rows_moved(ps) -> int:
    out = _u64(0)
    _check(load_library().ps_rows_moved(ps, C.byref(out)), "ps_rows_moved")
    return out.value


def ps_profile_start(ps, max_launches: int) -> None:
    _check(load_library().ps_profile_start(ps, max_launches), "ps_profile_start")


def ps_profile_stop(ps) -> dict:
    """{kernel name: (launches, total microseconds)} in first-launch order."""
    buf = C.create_string_buffer(1 << 16)
    _check(load_library().ps_profile_stop(ps, buf, len(buf)), "ps_profile_stop")
    out = {}
    for line in buf.value.decode().splitlines():
        name, launches, us = line.rsplit(" ", 2)
        out[name] = (int(launches), float(us))
    return out


def ps_status_string(code: int) -> str:
    return load_library().ps_status_string(code).decode()


def ps_dsgd_epoch_mf(ps, d_i, d_j, d_v, h_offsets, rows, cols, batch, lr, lam, d_loss_accum=None):
    """h_offsets: CPU int64 tensor of N * N + 1 stratum boundaries."""
    _check(load_library().ps_dsgd_epoch_mf(ps, _dptr(d_i, _U32), _dptr(d_j, _U32), _dptr(d_v, _F32), _hptr(h_offsets, _U64),
                                           rows, cols, batch, lr, lam, _dptr(d_loss_accum, _F64), _stream()),
           "ps_dsgd_epoch_mf")


def ps_keymap_query_bytes(capacity: int, max_batch_keys: int) -> int:
    out = _sz(0)
    _check(load_library().ps_keymap_query_bytes(capacity, max_batch_keys, C.byref(out)), "ps_keymap_query_bytes")
    return out.value


def ps_keymap_create(capacity: int, max_batch_keys: int, d_mem, device: int = 0):
    h = _vp()
    _check(load_library().ps_keymap_create(capacity, max_batch_keys, _dptr(d_mem), d_mem.numel() * d_mem.element_size(),
                                           device, _stream(), C.byref(h)), "ps_keymap_create")
    return h


def ps_keymap_destroy(m):
    _check(load_library().ps_keymap_destroy(m), "ps_keymap_destroy")


def ps_keymap_insert(m, d_sparse, d_dense):
    _check(load_library().ps_keymap_insert(m, _dptr(d_sparse, _U64), d_sparse.numel(), _dptr(d_dense, _U64), _stream()),
           "ps_keymap_insert")


def ps_keymap_lookup(m, d_sparse, d_dense):
    _check(load_library().ps_keymap_lookup(m, _dptr(d_sparse, _U64), d_sparse.numel(), _dptr(d_dense, _U64), _stream()),
           "ps_keymap_lookup")


def ps_keymap_sync(m):
    """(latched status code, number of dense keys handed out so far)."""
    size = _u64(0)
    code = load_library().ps_keymap_sync(m, _stream(), C.byref(size))
    return code, size.value


def ps_keymap_launch_count(m) -> int:
    return load_library().ps_keymap_launch_count(m)


class KeyMap:
    """A sparse-key map whose device memory is a torch tensor (memory only)."""

    def __init__(self, capacity: int, max_batch_keys: int = 1 << 20, device: int = 0):
        self.device = torch.device("cuda", device)
        n = ps_keymap_query_bytes(capacity, max_batch_keys)
        with torch.cuda.device(self.device):
            self.mem = torch.empty((n + 7) // 8, dtype=torch.int64, device=self.device)
            self.h = ps_keymap_create(capacity, max_batch_keys, self.mem, device)

    def insert(self, sparse):
        out = torch.empty(sparse.numel(), dtype=torch.int64, device=self.device)
        ps_keymap_insert(self.h, sparse, out)
        return out

    def lookup(self, sparse):
        out = torch.empty(sparse.numel(), dtype=torch.int64, device=self.device)
        ps_keymap_lookup(self.h, sparse, out)
        return out

    def sync(self):
        return ps_keymap_sync(self.h)

    def close(self):
        if getattr(self, "h", None):
            ps_keymap_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


# ---- convenience: torch-owned buffers around one handle -------------------------------
class Store:
    """A parameter store whose device buffers are torch tensors (memory only; no torch compute)."""

    def __init__(self, num_keys: int, row_len: int, num_workers: int = 1, slots_per_part: int | None = None,
                 max_batch_keys: int = 1 << 20, device: int = 0):
        load_library()
        if not torch.cuda.is_available():
            raise RuntimeError("a CUDA device is required: this library has no CPU path")
        part = (num_keys + num_workers - 1) // num_workers
        self.cfg = ps_config_t(num_keys, row_len, num_workers, part if slots_per_part is None else slots_per_part,
                               device)
        self.K, self.L, self.N, self.S = num_keys, row_len, num_workers, self.cfg.slots_per_part
        self.max_batch_keys = max_batch_keys
        sz = ps_query_sizes(self.cfg, max_batch_keys)
        self.sizes = sz
        dev = torch.device("cuda", device)
        self.device = dev
        with torch.cuda.device(dev):
            self.store = torch.zeros(sz.store_bytes // 4, dtype=torch.float32, device=dev)
            self.table = torch.empty(sz.table_bytes // 8, dtype=torch.int64, device=dev)
            self.freelists = torch.empty((sz.freelist_bytes + 7) // 8, dtype=torch.int64, device=dev)
            self.workspace = torch.empty((sz.workspace_bytes + 7) // 8, dtype=torch.int64, device=dev)
            self.loss = torch.zeros(1, dtype=torch.float64, device=dev)
            self.h = ps_create(self.cfg, self.store, self.table, self.freelists, self.workspace, max_batch_keys)
            ps_init_range_partition(self.h)

    def close(self):
        if getattr(self, "h", None):
            ps_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def sync(self, check: bool = True) -> int:
        code = ps_sync(self.h)
        if check and code != PS_OK:
            raise PSError(code, "ps_sync")
        return code

    def set_rows(self, keys, vals):
        ps_set_rows(self.h, keys, vals.contiguous())

    def set_all_rows(self, vals, chunk: int = 1 << 22):
        """Rows of keys 0..K-1 from a [K, L] tensor (any device), in chunks."""
        for s in range(0, self.K, chunk):
            c = min(chunk, self.K - s)
            keys = torch.arange(s, s + c, dtype=torch.int64, device=self.device)
            ps_set_rows(self.h, keys, vals[s:s + c].to(self.device, non_blocking=False).contiguous())
        torch.cuda.synchronize(self.device)

    def pull(self, keys):
        out = torch.empty((keys.numel(), self.L), dtype=torch.float32, device=self.device)
        ps_pull(self.h, keys, out)
        return out

    def push(self, keys, updates):
        ps_push(self.h, keys, updates)

    def localize(self, worker, keys):
        ps_localize(self.h, worker, keys)

    def export(self, rows=True, table=True):
        """(rows_by_key [K, L] | None, owner [K] | None, slot [K] | None) as CPU tensors."""
        r = torch.empty((self.K, self.L), dtype=torch.float32) if rows else None
        o = torch.empty(self.K, dtype=torch.int32) if table else None
        s = torch.empty(self.K, dtype=torch.int32) if table else None
        ps_export(self.h, r, o, s)
        return r, o, s

    def export_freelists(self):
        st = torch.empty((self.N, self.S), dtype=torch.int32)
        tp = torch.empty(self.N, dtype=torch.int64)
        ps_export_freelists(self.h, st, tp)
        return st, tp

    def launch_count(self) -> int:
        return ps_launch_count(self.h)
