"""ctypes binding of libemoe.so: argument marshalling only.

Every step of the re-layout runs inside the library's CUDA kernels; this module
converts Python objects to the C structs of include/emoe.h and back.  It fails
loudly if the library cannot be loaded: there is no CPU fallback.
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence

import numpy as np

from . import build as _build

PHASE_EXPERTS, PHASE_ATTN, PHASE_KV = 0, 1, 2
PHASE_STEP = 3   # num_launches only: one reshard_step call
SIDE_OLD, SIDE_NEW = 0, 1
PLAN_HOST_ONLY = 1
PLAN_HOST_STEP = 2
LAYOUT_FUSED_W13 = 4
LAYOUT_KV_HEAD_MAJOR = 8
LAYOUT_FUSED_QKV = 16
MAX_RANKS = 64

_i32, _u32, _u64, _vp = ctypes.c_int32, ctypes.c_uint32, ctypes.c_uint64, ctypes.c_void_p
_i32p = ctypes.POINTER(ctypes.c_int32)


class EmoeError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__("libemoe: %s (status %d)" % (what, code))
        self.code = code


class _Shape(ctypes.Structure):
    _fields_ = [(n, _i32) for n in ("n_layers", "n_routed", "n_shared", "d_model", "d_ff",
                                    "n_q_heads", "n_kv_heads", "head_dim", "kv_block_tokens",
                                    "elem_bytes")]


class _Config(ctypes.Structure):
    _fields_ = [("ep", _i32), ("tp", _i32), ("place_off", _i32p), ("place_ids", _i32p),
                ("kv_num_blocks", _i32), ("n_seqs", _i32), ("max_blocks", _i32),
                ("seq_lens", _i32p), ("block_table", _i32p)]


class _PlanOptions(ctypes.Structure):
    _fields_ = [("expert_scale_bytes", ctypes.c_int64), ("attn_new_replicas", ctypes.c_int64),
                ("reserved", ctypes.c_int64 * 6)]


class _Segment(ctypes.Structure):
    _fields_ = [("src_off", _u64), ("dst_off", _u64), ("run_bytes", _u64), ("src_pitch", _u64),
                ("dst_pitch", _u64), ("n_runs", _u32), ("src_rank", _u32), ("dst_rank", _u32),
                ("group", _u32)]


class _Tuning(ctypes.Structure):
    _fields_ = [("max_ctas", _i32), ("bulk_tile_bytes", _i32), ("bulk_stages", _i32),
                ("path", _i32), ("kv_mode", _i32), ("bulk_hints", _i32), ("kv_order", _i32),
                ("unit_order", _i32), ("wait_limit_us", _i32), ("bw_limit_gbs", _i32),
                ("bulk_min_run", _i32), ("serial", _i32)]


class _VmmStats(ctypes.Structure):
    _fields_ = [(n, _u64) for n in ("slabs_remapped", "slabs_copied", "bytes_copied", "bytes_read",
                                    "slab_bytes", "matrix_bytes", "physical_bytes")] + \
               [(n, ctypes.c_double) for n in ("map_ms", "alloc_ms", "access_ms", "copy_ms", "unmap_ms",
                                               "total_ms")]


SEGMENT_DTYPE = np.dtype([("src_off", "<u8"), ("dst_off", "<u8"), ("run_bytes", "<u8"),
                          ("src_pitch", "<u8"), ("dst_pitch", "<u8"), ("n_runs", "<u4"),
                          ("src_rank", "<u4"), ("dst_rank", "<u4"), ("group", "<u4")])

EXPORTS = ("emoe_plan_create", "emoe_plan_create_ex", "emoe_reshard_experts", "emoe_reshard_attn", "emoe_reshard_kv",
           "emoe_reshard_kv_static", "emoe_reshard_step", "emoe_plan_create_inplace",
           "emoe_plan_slot_table", "emoe_reshard_experts_inplace",
           "emoe_reshard_step_host", "emoe_plan_destroy", "emoe_plan_num_ranks",
           "emoe_plan_arena_bytes", "emoe_plan_stats", "emoe_plan_num_launches", "emoe_plan_launch_work",
           "emoe_plan_phase_is_identity",
           "emoe_plan_segments",
           "emoe_plan_device_status", "emoe_plan_clear_device_status", "emoe_plan_set_tuning",
           "emoe_segments_validate", "emoe_plan_validate",
           "emoe_strerror",
           "emoe_plan_cache_create", "emoe_plan_cache_get", "emoe_plan_cache_stats", "emoe_plan_cache_destroy",
           "emoe_kv_compact_table", "emoe_place_min_transfer", "emoe_plan_set_local_rank", "emoe_ipc_export", "emoe_ipc_open", "emoe_ipc_close",
           "emoe_vmm_create", "emoe_vmm_reshard", "emoe_vmm_dry_run", "emoe_vmm_num_ranks", "emoe_vmm_arena",
           "emoe_vmm_write", "emoe_vmm_read", "emoe_vmm_destroy",
           "emoe_vmm_slots_create", "emoe_vmm_slots_reshard", "emoe_vmm_slots_info", "emoe_vmm_slots_write",
           "emoe_vmm_slots_read", "emoe_vmm_slots_destroy")

_lib: Optional[ctypes.CDLL] = None


def library_path() -> str:
    return _build.OUT


def lib() -> ctypes.CDLL:
    """Loads libemoe.so, building it first if the sources are newer.  Raises if that fails."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.OUT
    if _build.is_stale():
        if _build.have_nvcc():
            _build.build()      # a failed compile raises: a stale binary is never used in its place
        elif not os.path.exists(path):
            raise RuntimeError("libemoe.so is missing and there is no nvcc to build it with")
        # no nvcc on this machine: the shipped binary is all there is
    L = ctypes.CDLL(path)
    PP = ctypes.POINTER(_vp)
    L.emoe_plan_create.restype = _i32
    L.emoe_plan_create.argtypes = [ctypes.POINTER(_Shape), ctypes.POINTER(_Config),
                                   ctypes.POINTER(_Config), _u32, ctypes.POINTER(_vp)]
    L.emoe_plan_create_ex.restype = _i32
    L.emoe_plan_create_ex.argtypes = [ctypes.POINTER(_Shape), ctypes.POINTER(_Config),
                                      ctypes.POINTER(_Config), _u32, ctypes.POINTER(_PlanOptions),
                                      ctypes.POINTER(_vp)]
    for name in ("emoe_reshard_experts", "emoe_reshard_attn", "emoe_reshard_kv",
                 "emoe_reshard_kv_static"):
        f = getattr(L, name)
        f.restype = _i32
        f.argtypes = [_vp, PP, PP, _vp]
    L.emoe_plan_create_inplace.restype = _i32
    L.emoe_plan_create_inplace.argtypes = [ctypes.POINTER(_Shape), _i32, _i32p, _i32p, _i32, _i32p, _i32p,
                                           _i32p, _u32, ctypes.POINTER(_vp)]
    L.emoe_plan_slot_table.restype = _i32
    L.emoe_plan_slot_table.argtypes = [_vp, _i32, _i32p, _i32, _i32p]
    L.emoe_reshard_experts_inplace.restype = _i32
    L.emoe_reshard_experts_inplace.argtypes = [_vp, PP, _vp]
    L.emoe_reshard_step.restype = _i32
    L.emoe_reshard_step.argtypes = [_vp, ctypes.POINTER(PP), ctypes.POINTER(PP), _vp]
    L.emoe_reshard_step_host.restype = _i32
    L.emoe_reshard_step_host.argtypes = [_vp, ctypes.POINTER(PP), ctypes.POINTER(PP),
                                         ctypes.POINTER(PP), ctypes.POINTER(PP), _vp]
    L.emoe_plan_destroy.restype = None
    L.emoe_plan_destroy.argtypes = [_vp]
    L.emoe_plan_num_ranks.restype = _i32
    L.emoe_plan_num_ranks.argtypes = [_vp, _i32, _i32, ctypes.POINTER(_i32)]
    L.emoe_plan_arena_bytes.restype = _i32
    L.emoe_plan_arena_bytes.argtypes = [_vp, _i32, _i32, _i32, ctypes.POINTER(_u64)]
    L.emoe_plan_stats.restype = _i32
    L.emoe_plan_stats.argtypes = [_vp, _i32] + [ctypes.POINTER(_u64)] * 3
    L.emoe_plan_num_launches.restype = _i32
    L.emoe_plan_num_launches.argtypes = [_vp, _i32, ctypes.POINTER(_i32)]
    L.emoe_plan_phase_is_identity.restype = _i32
    L.emoe_plan_phase_is_identity.argtypes = [_vp, _i32]
    L.emoe_plan_launch_work.restype = _i32
    L.emoe_plan_launch_work.argtypes = [_vp, _i32] + [ctypes.POINTER(_u64)] * 3
    L.emoe_plan_segments.restype = _i32
    L.emoe_plan_segments.argtypes = [_vp, _i32, _vp, _u64, ctypes.POINTER(_u64)]
    L.emoe_plan_device_status.restype = _i32
    L.emoe_plan_device_status.argtypes = [_vp, ctypes.POINTER(_i32)]
    L.emoe_segments_validate.restype = _i32
    L.emoe_segments_validate.argtypes = [_vp, _u64, ctypes.POINTER(_u64), _i32, ctypes.POINTER(_u64), _i32,
                                         _i32, ctypes.POINTER(_u64)]
    L.emoe_plan_validate.restype = _i32
    L.emoe_plan_validate.argtypes = [_vp, _i32p, ctypes.POINTER(_u64)]
    L.emoe_plan_clear_device_status.restype = _i32
    L.emoe_plan_clear_device_status.argtypes = [_vp]
    L.emoe_plan_set_tuning.restype = _i32
    L.emoe_plan_set_tuning.argtypes = [_vp, ctypes.POINTER(_Tuning)]
    L.emoe_plan_cache_create.restype = _i32
    L.emoe_plan_cache_create.argtypes = [_i32, ctypes.POINTER(_vp)]
    L.emoe_plan_cache_get.restype = _i32
    L.emoe_plan_cache_get.argtypes = [_vp, ctypes.POINTER(_Shape), ctypes.POINTER(_Config),
                                      ctypes.POINTER(_Config), _u32, ctypes.POINTER(_PlanOptions),
                                      ctypes.POINTER(_vp), _i32p]
    L.emoe_plan_cache_stats.restype = _i32
    L.emoe_plan_cache_stats.argtypes = [_vp] + [ctypes.POINTER(_u64)] * 3 + [_i32p]
    L.emoe_plan_cache_destroy.restype = None
    L.emoe_plan_cache_destroy.argtypes = [_vp]
    L.emoe_kv_compact_table.restype = _i32
    L.emoe_kv_compact_table.argtypes = [_i32, _i32, _i32, _i32p, _i32, _i32p, _i32, _i32p, _i32p, _i32p]
    L.emoe_place_min_transfer.restype = _i32
    L.emoe_place_min_transfer.argtypes = [_i32, ctypes.POINTER(_Config), _i32, _i32p, _i32p, _i32p]
    L.emoe_plan_set_local_rank.restype = _i32
    L.emoe_plan_set_local_rank.argtypes = [_vp, _i32]
    L.emoe_ipc_export.restype = _i32
    L.emoe_ipc_export.argtypes = [_vp, ctypes.c_char_p, ctypes.POINTER(_u64)]
    L.emoe_ipc_open.restype = _i32
    L.emoe_ipc_open.argtypes = [ctypes.c_char_p, ctypes.POINTER(_vp)]
    L.emoe_ipc_close.restype = _i32
    L.emoe_ipc_close.argtypes = [_vp]
    L.emoe_vmm_create.restype = _i32
    L.emoe_vmm_create.argtypes = [ctypes.POINTER(_Shape), ctypes.POINTER(_Config), ctypes.POINTER(_vp)]
    L.emoe_vmm_reshard.restype = _i32
    L.emoe_vmm_reshard.argtypes = [_vp, ctypes.POINTER(_Config), _vp, ctypes.POINTER(_VmmStats)]
    L.emoe_vmm_dry_run.restype = _i32
    L.emoe_vmm_dry_run.argtypes = [ctypes.POINTER(_Shape), ctypes.POINTER(_Config),
                                   ctypes.POINTER(_Config), _u64, ctypes.POINTER(_VmmStats)]
    L.emoe_vmm_num_ranks.restype = _i32
    L.emoe_vmm_num_ranks.argtypes = [_vp, ctypes.POINTER(_i32)]
    L.emoe_vmm_arena.restype = _i32
    L.emoe_vmm_arena.argtypes = [_vp, _i32, ctypes.POINTER(_vp), ctypes.POINTER(_u64),
                                 ctypes.POINTER(_u64), ctypes.POINTER(_u64), ctypes.POINTER(_i32)]
    for name in ("emoe_vmm_write", "emoe_vmm_read"):
        f = getattr(L, name)
        f.restype = _i32
        f.argtypes = [_vp, _i32, _vp, _vp]
    L.emoe_vmm_destroy.restype = None
    L.emoe_vmm_destroy.argtypes = [_vp]
    L.emoe_vmm_slots_create.restype = _i32
    L.emoe_vmm_slots_create.argtypes = [ctypes.POINTER(_Shape), _i32, _i32p, _i32p, _i32, ctypes.POINTER(_vp)]
    L.emoe_vmm_slots_reshard.restype = _i32
    L.emoe_vmm_slots_reshard.argtypes = [_vp, _i32, _i32p, _i32p, _i32p, _vp, ctypes.POINTER(_VmmStats)]
    L.emoe_vmm_slots_info.restype = _i32
    L.emoe_vmm_slots_info.argtypes = [_vp, _i32, ctypes.POINTER(_vp), ctypes.POINTER(_u64), _i32p, _i32p, _i32,
                                      _i32p, ctypes.POINTER(ctypes.c_int64)]
    for name in ("emoe_vmm_slots_write", "emoe_vmm_slots_read"):
        f = getattr(L, name)
        f.restype = _i32
        f.argtypes = [_vp, _i32, _i32, _vp, _vp]
    L.emoe_vmm_slots_destroy.restype = None
    L.emoe_vmm_slots_destroy.argtypes = [_vp]
    L.emoe_strerror.restype = ctypes.c_char_p
    L.emoe_strerror.argtypes = [_i32]
    _lib = L
    return L


def strerror(code: int) -> str:
    return lib().emoe_strerror(code).decode()


def _check(code: int) -> None:
    if code != 0:
        raise EmoeError(code, strerror(code))


def _i32arr(x) -> np.ndarray:
    return np.ascontiguousarray(x, dtype=np.int32)


def _make_config(cfg, keep: list) -> _Config:
    """cfg: object with ep, tp, placement, kv_num_blocks, seq_lens, block_table."""
    off = np.zeros(len(cfg.placement) + 1, dtype=np.int32)
    off[1:] = np.cumsum([len(p) for p in cfg.placement])
    ids = _i32arr([e for p in cfg.placement for e in p])
    if ids.size == 0:
        ids = np.zeros(1, dtype=np.int32)
    sl = _i32arr(cfg.seq_lens)
    bt = _i32arr(cfg.block_table)
    n_seqs = int(sl.size)
    max_blocks = int(bt.shape[1]) if bt.ndim == 2 and n_seqs else 0
    if sl.size == 0:
        sl = np.zeros(1, dtype=np.int32)
    if bt.size == 0:
        bt = np.zeros(1, dtype=np.int32)
    keep += [off, ids, sl, bt]
    p = lambda a: a.ctypes.data_as(_i32p)
    return _Config(cfg.ep, cfg.tp, p(off), p(ids), cfg.kv_num_blocks, n_seqs, max_blocks,
                   p(sl), p(bt))


def _ptr_array(items: Sequence) -> ctypes.Array:
    """Device (or host) addresses from ints, torch tensors or numpy arrays."""
    vals = []
    for x in items:
        if x is None:
            vals.append(0)
        elif isinstance(x, int):
            vals.append(x)
        elif hasattr(x, "data_ptr"):
            vals.append(x.data_ptr())
        elif isinstance(x, np.ndarray):
            vals.append(x.ctypes.data)
        else:
            raise TypeError("cannot take the address of %r" % type(x))
    return (_vp * max(len(vals), 1))(*vals)


def _stream_handle(stream) -> int:
    if stream is None:
        return 0
    if isinstance(stream, int):
        return stream
    return int(stream.cuda_stream)


class Plan:
    """A scale-step plan: emoe_plan_create ... emoe_plan_destroy."""

    def __init__(self, shape, old_cfg, new_cfg, host_only: bool = False, host_step: bool = False,
                 fused_w13: bool = False, kv_head_major: bool = False, fused_qkv: bool = False,
                 attn_replicas: int = 1):
        self._h = _vp()
        keep: list = []
        sh = _Shape(shape.n_layers, shape.n_routed, shape.n_shared, shape.d_model, shape.d_ff,
                    shape.n_q_heads, shape.n_kv_heads, shape.head_dim, shape.kv_block_tokens,
                    shape.elem_bytes)
        co, cn = _make_config(old_cfg, keep), _make_config(new_cfg, keep)
        flags = ((PLAN_HOST_ONLY if host_only else 0) | (PLAN_HOST_STEP if host_step else 0)
                 | (LAYOUT_FUSED_W13 if fused_w13 else 0) | (LAYOUT_KV_HEAD_MAJOR if kv_head_major else 0)
                 | (LAYOUT_FUSED_QKV if fused_qkv else 0))
        scale = int(getattr(shape, "expert_scale_bytes", 0) or 0)
        if scale or attn_replicas > 1:     # scale tensors with the matrices / several new DP replicas
            opt = _PlanOptions(scale, attn_replicas)
            _check(lib().emoe_plan_create_ex(ctypes.byref(sh), ctypes.byref(co), ctypes.byref(cn), flags,
                                             ctypes.byref(opt), ctypes.byref(self._h)))
        else:
            _check(lib().emoe_plan_create(ctypes.byref(sh), ctypes.byref(co), ctypes.byref(cn), flags,
                                          ctypes.byref(self._h)))
        self.host_only = host_only

    # -- life cycle
    _owned = True     # False: the handle belongs to a PlanCache

    def close(self) -> None:
        if self._h:
            if self._owned:
                lib().emoe_plan_destroy(self._h)
            self._h = _vp()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *a):
        self.close()

    # -- queries
    def num_ranks(self, phase: int, side: int) -> int:
        n = _i32()
        _check(lib().emoe_plan_num_ranks(self._h, phase, side, ctypes.byref(n)))
        return n.value

    def arena_bytes(self, phase: int, side: int) -> List[int]:
        out = []
        for r in range(self.num_ranks(phase, side)):
            b = _u64()
            _check(lib().emoe_plan_arena_bytes(self._h, phase, side, r, ctypes.byref(b)))
            out.append(b.value)
        return out

    def stats(self, phase: int) -> dict:
        a, b, c = _u64(), _u64(), _u64()
        _check(lib().emoe_plan_stats(self._h, phase, ctypes.byref(a), ctypes.byref(b),
                                     ctypes.byref(c)))
        return dict(bytes_moved=a.value, bytes_read=b.value, n_segments=c.value)

    def num_launches(self, phase: int) -> int:
        n = _i32()
        _check(lib().emoe_plan_num_launches(self._h, phase, ctypes.byref(n)))
        return n.value

    def phase_is_identity(self, phase: int) -> bool:
        """True when the phase moves every byte onto its own place: src arenas may then be
        passed as dst arenas and nothing is launched (the zero-copy case, Sec. 5.2)."""
        r = lib().emoe_plan_phase_is_identity(self._h, phase)
        if r < 0:
            raise EmoeError(1, strerror(1))
        return bool(r)

    def launch_work(self, phase: int) -> dict:
        """Work items per kind of kernel for one call of this phase (PHASE_STEP: a whole step)."""
        a, b, c = _u64(), _u64(), _u64()
        _check(lib().emoe_plan_launch_work(self._h, phase, ctypes.byref(a), ctypes.byref(b),
                                           ctypes.byref(c)))
        return dict(ring_units=a.value, vector_units=b.value, kv_tiles=c.value)

    def segments(self, phase: int) -> np.ndarray:
        n = _u64()
        _check(lib().emoe_plan_segments(self._h, phase, None, 0, ctypes.byref(n)))
        out = np.zeros(n.value, dtype=SEGMENT_DTYPE)
        if n.value:
            _check(lib().emoe_plan_segments(self._h, phase, out.ctypes.data_as(_vp), n.value,
                                            ctypes.byref(n)))
        return out

    def validate(self) -> None:
        """Host-side bounds and race check of the plan's segments; raises EmoeError (status 12)
        naming the phase and segment if a run leaves its arena or two runs write one byte."""
        ph, seg = _i32(-1), _u64(0)
        code = lib().emoe_plan_validate(self._h, ctypes.byref(ph), ctypes.byref(seg))
        if code != 0:
            raise EmoeError(code, "%s (phase %d, segment %d)" % (strerror(code), ph.value, seg.value))

    def device_status(self) -> int:
        s = _i32()
        _check(lib().emoe_plan_device_status(self._h, ctypes.byref(s)))
        return s.value

    def clear_device_status(self) -> None:
        _check(lib().emoe_plan_clear_device_status(self._h))

    def set_tuning(self, max_ctas: int = 0, bulk_tile_bytes: int = 0, bulk_stages: int = 0,
                   path: int = 0, kv_mode: int = 0, bulk_hints: int = 0, kv_order: int = 0,
                   unit_order: int = 0, wait_limit_us: int = 0, bw_limit_gbs: int = 0,
                   bulk_min_run: int = 0, serial: int = 0) -> None:
        t = _Tuning(max_ctas, bulk_tile_bytes, bulk_stages, path, kv_mode, bulk_hints, kv_order,
                    unit_order, wait_limit_us, bw_limit_gbs, bulk_min_run, serial)
        _check(lib().emoe_plan_set_tuning(self._h, ctypes.byref(t)))

    def set_local_rank(self, rank: int) -> None:
        """From now on write only the destination arenas of new-rank index `rank` (-1: all)."""
        _check(lib().emoe_plan_set_local_rank(self._h, rank))

    # -- the hot path
    def _run(self, fn, src, dst, stream) -> None:
        _check(fn(self._h, _ptr_array(src), _ptr_array(dst), _stream_handle(stream)))

    def reshard_experts(self, src, dst, stream=None) -> None:
        self._run(lib().emoe_reshard_experts, src, dst, stream)

    def reshard_attn(self, src, dst, stream=None) -> None:
        self._run(lib().emoe_reshard_attn, src, dst, stream)

    def reshard_kv(self, src, dst, stream=None) -> None:
        self._run(lib().emoe_reshard_kv, src, dst, stream)

    def reshard_kv_static(self, src, dst, stream=None) -> None:
        """emoe_reshard_kv for callers that may not allocate device memory (a process
        whose HBM is fully owned by a memory daemon, a section that cannot afford the
        implicit synchronisation of cudaMalloc).  Works on host-only plans; the block
        pair list goes into a fixed 512 KiB array of the library image, shared by all
        calls on the device, so calls that may overlap on the GPU must be serialised.
        Make the first call on a device outside stream capture."""
        self._run(lib().emoe_reshard_kv_static, src, dst, stream)

    def reshard_step(self, src, dst, stream=None) -> None:
        """All three phases as one set of launches.  src / dst: three lists (experts, attn,
        kv) of per-rank device buffers."""
        PP = ctypes.POINTER(_vp)
        arrs = [_ptr_array(g) for g in list(src) + list(dst)]
        pack = lambda a: (PP * 3)(*[ctypes.cast(x, PP) for x in a])
        _check(lib().emoe_reshard_step(self._h, pack(arrs[:3]), pack(arrs[3:]), _stream_handle(stream)))

    def reshard_step_host(self, h_src, h_dst, d_src, d_dst, stream=None) -> None:
        """Each argument: three lists (experts, attn, kv) of per-rank buffers."""
        PP = ctypes.POINTER(_vp)
        keep = []

        def pack(groups):
            arrs = [_ptr_array(g) for g in groups]
            keep.extend(arrs)
            return (PP * 3)(*[ctypes.cast(a, PP) for a in arrs])

        _check(lib().emoe_reshard_step_host(self._h, pack(h_src), pack(h_dst), pack(d_src),
                                            pack(d_dst), _stream_handle(stream)))


def _plan_flags(host_only=False, host_step=False, fused_w13=False, kv_head_major=False, fused_qkv=False):
    return ((PLAN_HOST_ONLY if host_only else 0) | (PLAN_HOST_STEP if host_step else 0)
            | (LAYOUT_FUSED_W13 if fused_w13 else 0) | (LAYOUT_KV_HEAD_MAJOR if kv_head_major else 0)
            | (LAYOUT_FUSED_QKV if fused_qkv else 0))


class PlanCache:
    """emoe_plan_cache_*: plans of a scaling sequence, kept and handed out again when the
    same (shape, old, new, flags) pair comes back.  The cache owns its plans: the Plan
    objects returned by get() must not outlive it, and at most `capacity` of them stay
    valid (the least recently used one is destroyed when one more is inserted)."""

    def __init__(self, capacity: int = 16):
        self._h = _vp()
        _check(lib().emoe_plan_cache_create(capacity, ctypes.byref(self._h)))

    def get(self, shape, old_cfg, new_cfg, **flags):
        """(plan, hit)"""
        keep: list = []
        sh = _Shape(shape.n_layers, shape.n_routed, shape.n_shared, shape.d_model, shape.d_ff,
                    shape.n_q_heads, shape.n_kv_heads, shape.head_dim, shape.kv_block_tokens,
                    shape.elem_bytes)
        co, cn = _make_config(old_cfg, keep), _make_config(new_cfg, keep)
        scale = int(getattr(shape, "expert_scale_bytes", 0) or 0)
        replicas = int(flags.pop("attn_replicas", 1))
        opt = _PlanOptions(scale, replicas)
        h, hit = _vp(), _i32()
        _check(lib().emoe_plan_cache_get(self._h, ctypes.byref(sh), ctypes.byref(co), ctypes.byref(cn),
                                         _plan_flags(**flags), ctypes.byref(opt) if scale or replicas > 1 else None,
                                         ctypes.byref(h), ctypes.byref(hit)))
        plan = Plan.__new__(Plan)
        plan._h, plan._owned, plan.host_only = h, False, bool(flags.get("host_only"))
        return plan, bool(hit.value)

    def stats(self) -> dict:
        a, b, c, n = _u64(), _u64(), _u64(), _i32()
        _check(lib().emoe_plan_cache_stats(self._h, ctypes.byref(a), ctypes.byref(b), ctypes.byref(c),
                                           ctypes.byref(n)))
        return dict(hits=a.value, misses=b.value, evictions=c.value, size=n.value)

    def close(self) -> None:
        if self._h:
            lib().emoe_plan_cache_destroy(self._h)
            self._h = _vp()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *a):
        self.close()


def kv_compact_table(block_tokens: int, seq_lens, nb_new: int, in_use=(), max_blocks: Optional[int] = None,
                     old_table=None):
    """Destination block table [n_seqs, max_blocks] that packs the sequences' blocks into the
    lowest free blocks of a pool of nb_new blocks (in_use: ids already taken there), in table
    order or - with old_table - in the order of the blocks' old physical ids."""
    sl = _i32arr(seq_lens)
    need = [-(-int(n) // block_tokens) for n in sl]
    mb = max_blocks if max_blocks is not None else max(need, default=0)
    old = None
    if old_table is not None:
        old = np.full((len(sl), max(mb, 1)), -1, dtype=np.int32)
        src = np.asarray(old_table, dtype=np.int32).reshape(len(sl), -1)[:, :mb]
        old[:, :src.shape[1]] = src
    out = np.full((len(sl), max(mb, 1)), -1, dtype=np.int32)
    if mb == 0:
        return out[:, :0]
    used = _i32arr(list(in_use))
    n = _i32()
    _check(lib().emoe_kv_compact_table(block_tokens, len(sl), max(mb, 1),
                                       sl.ctypes.data_as(_i32p) if sl.size else None, nb_new,
                                       used.ctypes.data_as(_i32p) if used.size else None, int(used.size),
                                       old.ctypes.data_as(_i32p) if old is not None else None,
                                       out.ctypes.data_as(_i32p), ctypes.byref(n)))
    return out[:, :mb] if mb else out[:, :0]


class InplacePlan(Plan):
    """The expert step on capacity-strided arenas: emoe_plan_create_inplace.  old_slots: per
    old device a list of expert ids or -1 (free), as long as the device's capacity; want:
    per new device the experts it must hold; cap_new: capacity per new device."""

    def __init__(self, shape, old_slots, want, cap_new, host_only: bool = False):
        self._h = _vp()
        sh = _Shape(shape.n_layers, shape.n_routed, shape.n_shared, shape.d_model, shape.d_ff,
                    shape.n_q_heads, shape.n_kv_heads, shape.head_dim, shape.kv_block_tokens,
                    shape.elem_bytes)

        def csr(lists):
            off = np.zeros(len(lists) + 1, dtype=np.int32)
            off[1:] = np.cumsum([len(x) for x in lists])
            ids = _i32arr([e for x in lists for e in x])
            return off, (ids if ids.size else np.zeros(1, dtype=np.int32))

        oo, oi = csr(old_slots)
        wo, wi = csr(want)
        cap = _i32arr(cap_new)
        p = lambda a: a.ctypes.data_as(_i32p)
        _check(lib().emoe_plan_create_inplace(ctypes.byref(sh), len(old_slots), p(oo), p(oi), len(want),
                                              p(cap), p(wo), p(wi), PLAN_HOST_ONLY if host_only else 0,
                                              ctypes.byref(self._h)))
        self.host_only = host_only
        self.n_ranks = len(want)
        self.caps = [len(t) for t in old_slots] + [int(c) for c in list(cap_new)[len(old_slots):]]

    def slot_tables(self):
        out = []
        for r in range(self.n_ranks):
            n = _i32()
            _check(lib().emoe_plan_slot_table(self._h, r, None, 0, ctypes.byref(n)))
            t = np.zeros(max(n.value, 1), dtype=np.int32)
            _check(lib().emoe_plan_slot_table(self._h, r, t.ctypes.data_as(_i32p), n.value, ctypes.byref(n)))
            out.append([int(x) for x in t[:n.value]])
        return out

    def reshard(self, arenas, stream=None) -> None:
        """arenas: one device buffer per device index, max(old devices, new devices) of them."""
        _check(lib().emoe_reshard_experts_inplace(self._h, _ptr_array(arenas), _stream_handle(stream)))


IPC_HANDLE_BYTES = 64


def segments_validate(segs: np.ndarray, arena_old, arena_new, must_tile: bool = False) -> int:
    """emoe_segments_validate on a SEGMENT_DTYPE array; returns -1 if the list passes, else the
    index of an offending segment."""
    segs = np.ascontiguousarray(segs, dtype=SEGMENT_DTYPE)
    ao = np.ascontiguousarray(arena_old, dtype=np.uint64)
    an = np.ascontiguousarray(arena_new, dtype=np.uint64)
    bad = _u64(0)
    u64p = ctypes.POINTER(_u64)
    code = lib().emoe_segments_validate(segs.ctypes.data_as(_vp), len(segs), ao.ctypes.data_as(u64p), len(ao),
                                        an.ctypes.data_as(u64p), len(an), int(must_tile), ctypes.byref(bad))
    if code == 0:
        return -1
    if code != 12:
        _check(code)
    return int(bad.value)


def ipc_export(device_ptr: int):
    """(handle bytes, offset) naming the allocation that holds device_ptr."""
    buf = ctypes.create_string_buffer(IPC_HANDLE_BYTES)
    off = _u64()
    _check(lib().emoe_ipc_export(device_ptr, buf, ctypes.byref(off)))
    return buf.raw, off.value


def ipc_open(handle: bytes) -> int:
    """Maps another process's allocation; returns its base address in this process."""
    base = _vp()
    _check(lib().emoe_ipc_open(handle, ctypes.byref(base)))
    return base.value


def ipc_close(base: int) -> None:
    _check(lib().emoe_ipc_close(base))


def _placement_config(placement, keep: list) -> _Config:
    off = np.zeros(len(placement) + 1, dtype=np.int32)
    off[1:] = np.cumsum([len(p) for p in placement])
    ids = _i32arr([e for p in placement for e in p])
    if ids.size == 0:
        ids = np.zeros(1, dtype=np.int32)
    keep += [off, ids]
    p = lambda a: a.ctypes.data_as(_i32p)
    return _Config(len(placement), 1, p(off), p(ids), 0, 0, 0, None, None)


def place_min_transfer(n_experts: int, old_placement, ep_new: int):
    """(new placement, experts kept): balanced, every expert once, as many experts as
    possible on a rank index that already holds them."""
    keep: list = []
    off = np.zeros(ep_new + 1, dtype=np.int32)
    ids = np.zeros(n_experts, dtype=np.int32)
    kept = _i32()
    _check(lib().emoe_place_min_transfer(n_experts, ctypes.byref(_placement_config(old_placement, keep)),
                                         ep_new, off.ctypes.data_as(_i32p), ids.ctypes.data_as(_i32p),
                                         ctypes.byref(kept)))
    return [[int(e) for e in ids[off[r]:off[r + 1]]] for r in range(ep_new)], kept.value


def vmm_dry_run(shape, old_placement, new_placement, slab_bytes: int) -> dict:
    """What VmmPool.reshard would re-map and copy, computed on the host (no CUDA call)."""
    keep: list = []
    sh = _Shape(shape.n_layers, shape.n_routed, shape.n_shared, shape.d_model, shape.d_ff,
                shape.n_q_heads, shape.n_kv_heads, shape.head_dim, shape.kv_block_tokens,
                shape.elem_bytes)
    st = _VmmStats()
    _check(lib().emoe_vmm_dry_run(ctypes.byref(sh), ctypes.byref(_placement_config(old_placement, keep)),
                                  ctypes.byref(_placement_config(new_placement, keep)), slab_bytes,
                                  ctypes.byref(st)))
    return {n: getattr(st, n) for n, _ in _VmmStats._fields_}


class VmmPool:
    """Paged expert store: emoe_vmm_create ... emoe_vmm_destroy.  `cfg` objects need
    `placement` (expert ids per rank) only."""

    def __init__(self, shape, cfg):
        self._h = _vp()
        self._keep: list = []
        sh = _Shape(shape.n_layers, shape.n_routed, shape.n_shared, shape.d_model, shape.d_ff,
                    shape.n_q_heads, shape.n_kv_heads, shape.head_dim, shape.kv_block_tokens,
                    shape.elem_bytes)
        _check(lib().emoe_vmm_create(ctypes.byref(sh), ctypes.byref(self._config(cfg)),
                                     ctypes.byref(self._h)))

    def _config(self, cfg) -> _Config:
        placement = cfg.placement if hasattr(cfg, "placement") else cfg
        self._keep = []
        return _placement_config(placement, self._keep)

    def close(self) -> None:
        if self._h:
            lib().emoe_vmm_destroy(self._h)
            self._h = _vp()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *a):
        self.close()

    def num_ranks(self) -> int:
        n = _i32()
        _check(lib().emoe_vmm_num_ranks(self._h, ctypes.byref(n)))
        return n.value

    def arena(self, rank: int) -> dict:
        base, b, s, m, n = _vp(), _u64(), _u64(), _u64(), _i32()
        _check(lib().emoe_vmm_arena(self._h, rank, ctypes.byref(base), ctypes.byref(b),
                                    ctypes.byref(s), ctypes.byref(m), ctypes.byref(n)))
        return dict(base=base.value or 0, bytes=b.value, slab_bytes=s.value, matrix_bytes=m.value,
                    n_slots=n.value)

    def write(self, rank: int, host_dense, stream=None) -> None:
        _check(lib().emoe_vmm_write(self._h, rank, _ptr_array([host_dense])[0], _stream_handle(stream)))

    def read(self, rank: int, host_dense, stream=None) -> None:
        _check(lib().emoe_vmm_read(self._h, rank, _ptr_array([host_dense])[0], _stream_handle(stream)))

    def reshard(self, new_cfg, stream=None) -> dict:
        st = _VmmStats()
        _check(lib().emoe_vmm_reshard(self._h, ctypes.byref(self._config(new_cfg)),
                                      _stream_handle(stream), ctypes.byref(st)))
        return {n: getattr(st, n) for n, _ in _VmmStats._fields_}


def _csr_i32(lists):
    off = np.zeros(len(lists) + 1, dtype=np.int32)
    off[1:] = np.cumsum([len(x) for x in lists])
    ids = _i32arr([e for x in lists for e in x])
    return off, (ids if ids.size else np.zeros(1, dtype=np.int32))


class VmmSlots:
    """Paged expert store with slot tables: emoe_vmm_slots_create ... _destroy.  slots: per
    device a list of expert ids or -1 (free), as long as the device's capacity."""

    def __init__(self, shape, slots, spare_slots: int = 0):
        self._h = _vp()
        self.shape = shape
        sh = _Shape(shape.n_layers, shape.n_routed, shape.n_shared, shape.d_model, shape.d_ff,
                    shape.n_q_heads, shape.n_kv_heads, shape.head_dim, shape.kv_block_tokens,
                    shape.elem_bytes)
        off, ids = _csr_i32(slots)
        p = lambda a: a.ctypes.data_as(_i32p)
        _check(lib().emoe_vmm_slots_create(ctypes.byref(sh), len(slots), p(off), p(ids), spare_slots,
                                           ctypes.byref(self._h)))

    def close(self) -> None:
        if self._h:
            lib().emoe_vmm_slots_destroy(self._h)
            self._h = _vp()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *a):
        self.close()

    def info(self) -> dict:
        n, spare, slab = _i32(), ctypes.c_int64(), _u64()
        _check(lib().emoe_vmm_slots_info(self._h, -1, None, ctypes.byref(slab), None, None, 0,
                                         ctypes.byref(n), ctypes.byref(spare)))
        return dict(n_ranks=n.value, spare_slabs=spare.value, slab_bytes=slab.value)

    def tables(self):
        out = []
        for r in range(self.info()["n_ranks"]):
            cap = _i32()
            _check(lib().emoe_vmm_slots_info(self._h, r, None, None, ctypes.byref(cap), None, 0, None, None))
            t = np.zeros(max(cap.value, 1), dtype=np.int32)
            _check(lib().emoe_vmm_slots_info(self._h, r, None, None, None, t.ctypes.data_as(_i32p), cap.value,
                                             None, None))
            out.append([int(x) for x in t[:cap.value]])
        return out

    def base(self, rank: int) -> int:
        b = _vp()
        _check(lib().emoe_vmm_slots_info(self._h, rank, ctypes.byref(b), None, None, None, 0, None, None))
        return b.value or 0

    def write_slot(self, rank: int, slot: int, host, stream=None) -> None:
        _check(lib().emoe_vmm_slots_write(self._h, rank, slot, _ptr_array([host])[0], _stream_handle(stream)))

    def read_slot(self, rank: int, slot: int, host, stream=None) -> None:
        _check(lib().emoe_vmm_slots_read(self._h, rank, slot, _ptr_array([host])[0], _stream_handle(stream)))

    def reshard(self, want, cap_new, stream=None) -> dict:
        off, ids = _csr_i32(want)
        cap = _i32arr(cap_new)
        p = lambda a: a.ctypes.data_as(_i32p)
        st = _VmmStats()
        _check(lib().emoe_vmm_slots_reshard(self._h, len(want), p(cap), p(off), p(ids), _stream_handle(stream),
                                            ctypes.byref(st)))
        return {n: getattr(st, n) for n, _ in _VmmStats._fields_}

