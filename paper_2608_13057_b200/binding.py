"""Thin ctypes binding of libtempo.so.  Argument marshalling only: every step runs in the CUDA kernels.

The functions carry the C-ABI names (see include/tempo.h).  Tensors are torch CUDA tensors used as
device memory; kernels are enqueued on torch's current stream.  There is no CPU fallback: importing
this module without the built library, or calling it with CPU tensors, raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_LIB_PATH = os.environ.get("TEMPO_LIB") or os.path.join(os.path.dirname(os.path.abspath(__file__)), "libtempo.so")

TEMPO_OK = 0
STATUS_BAD_ID, STATUS_BAD_TABLE, STATUS_CAPACITY, STATUS_TIMEOUT, STATUS_BAD_SCALE = 1, 2, 4, 8, 16

EXPORTS = (
    "tempo_version", "tempo_status_string", "tempo_m_cap_bound", "tempo_sf_bytes", "tempo_workspace_bytes",
    "tempo_packed_weight_bytes",
    "tempo_pack_weights", "tempo_count_dispatch", "tempo_count_dispatch_sampled", "tempo_permute_pad", "tempo_ffn_gate_up", "tempo_ffn_down",
    "tempo_grouped_ffn", "tempo_grouped_ffn_bounded", "tempo_grouped_ffn_static",
    "tempo_token_sf_bytes", "tempo_quantize_tokens", "tempo_grouped_ffn_gather", "tempo_unpermute_combine",
    "tempo_count_dispatch_masked", "tempo_permute_pad_masked", "tempo_grouped_ffn_masked",
    "tempo_packed_weight_bytes_bf16", "tempo_pack_weights_bf16", "tempo_permute_pad_bf16", "tempo_grouped_ffn_bf16",
)


class TempoShape(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("T", "k", "E", "G_max", "R_max", "d", "f", "M_cap")]


class TempoError(RuntimeError):
    pass


def _load() -> ctypes.CDLL:
    if not os.path.exists(_LIB_PATH):
        raise ImportError(f"{_LIB_PATH} is missing: build it with __graft_entry__.build() "
                          "(python -m paper_2608_13057_b200.build); there is no fallback path")
    lib = ctypes.CDLL(_LIB_PATH)
    for name in EXPORTS:
        getattr(lib, name)                      # fail loudly on a missing symbol
    lib.tempo_status_string.restype = ctypes.c_char_p
    for name in EXPORTS:
        if name != "tempo_status_string":
            getattr(lib, name).restype = ctypes.c_int
    return lib


_lib = _load()


def _ptr(t: Optional[torch.Tensor], dtype=None):
    if t is None:
        return ctypes.c_void_p(0)
    if not t.is_cuda:
        raise TempoError("expected a CUDA tensor (the library has no CPU path)")
    if not t.is_contiguous():
        raise TempoError("expected a contiguous tensor")
    if dtype is not None and t.dtype != dtype:
        raise TempoError(f"expected dtype {dtype}, got {t.dtype}")
    return ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(rc: int, what: str):
    if rc != TEMPO_OK:
        raise TempoError(f"{what}: {_lib.tempo_status_string(rc).decode()} ({rc})")


def make_shape(T, k, E, G_max, R_max, d, f, M_cap) -> TempoShape:
    return TempoShape(T, k, E, G_max, R_max, d, f, M_cap)


def tempo_version() -> int:
    return _lib.tempo_version()


def tempo_m_cap_bound(shape: TempoShape) -> int:
    out = ctypes.c_int32(0)
    _check(_lib.tempo_m_cap_bound(ctypes.byref(shape), ctypes.byref(out)), "tempo_m_cap_bound")
    return out.value


def tempo_sf_bytes(rows: int, cols: int) -> int:
    out = ctypes.c_size_t(0)
    _check(_lib.tempo_sf_bytes(ctypes.c_int32(rows), ctypes.c_int32(cols), ctypes.byref(out)), "tempo_sf_bytes")
    return out.value


def tempo_workspace_bytes(shape: TempoShape) -> int:
    out = ctypes.c_size_t(0)
    _check(_lib.tempo_workspace_bytes(ctypes.byref(shape), ctypes.byref(out)), "tempo_workspace_bytes")
    return out.value


def tempo_packed_weight_bytes(shape: TempoShape) -> int:
    out = ctypes.c_size_t(0)
    _check(_lib.tempo_packed_weight_bytes(ctypes.byref(shape), ctypes.byref(out)), "tempo_packed_weight_bytes")
    return out.value


def tempo_pack_weights(shape, w13_q, w13_s, w2_q, w2_s, packed, status):
    _check(_lib.tempo_pack_weights(ctypes.byref(shape), _ptr(w13_q, torch.uint8), _ptr(w13_s, torch.float32),
                                   _ptr(w2_q, torch.uint8), _ptr(w2_s, torch.float32), _ptr(packed, torch.uint8),
                                   _ptr(status, torch.int32), _stream()), "tempo_pack_weights")


def tempo_count_dispatch(shape, topk_ids, n_valid, replica_map, quota, cum_counts, counts, inst_count, inst_off,
                         pair_row, row_pair, tile_inst, m_pad, status):
    i32 = torch.int32
    _check(_lib.tempo_count_dispatch(ctypes.byref(shape), _ptr(topk_ids, i32), _ptr(n_valid, i32),
                                     _ptr(replica_map, i32), _ptr(quota, i32), _ptr(cum_counts, i32),
                                     _ptr(counts, i32), _ptr(inst_count, i32), _ptr(inst_off, i32),
                                     _ptr(pair_row, i32), _ptr(row_pair, i32), _ptr(tile_inst, i32),
                                     _ptr(m_pad, i32), _ptr(status, i32), _stream()), "tempo_count_dispatch")


def tempo_count_dispatch_sampled(shape, topk_ids, n_valid, replica_map, table, seed, layer, cum_counts, counts,
                                 inst_count, inst_off, pair_row, row_pair, tile_inst, m_pad, status):
    i32 = torch.int32
    _check(_lib.tempo_count_dispatch_sampled(ctypes.byref(shape), _ptr(topk_ids, i32), _ptr(n_valid, i32),
                                             _ptr(replica_map, i32), _ptr(table, torch.float32),
                                             ctypes.c_uint64(int(seed)), ctypes.c_uint32(int(layer)),
                                             _ptr(cum_counts, i32), _ptr(counts, i32), _ptr(inst_count, i32),
                                             _ptr(inst_off, i32), _ptr(pair_row, i32), _ptr(row_pair, i32),
                                             _ptr(tile_inst, i32), _ptr(m_pad, i32), _ptr(status, i32), _stream()),
           "tempo_count_dispatch_sampled")


def tempo_permute_pad(shape, x_bf16, row_pair, m_pad, a_q, a_sf, status, pair_row=None):
    _check(_lib.tempo_permute_pad(ctypes.byref(shape), _ptr(x_bf16, torch.bfloat16), _ptr(row_pair, torch.int32),
                                  _ptr(pair_row, torch.int32),
                                  _ptr(m_pad, torch.int32), _ptr(a_q, torch.uint8), _ptr(a_sf, torch.uint8),
                                  _ptr(status, torch.int32), _stream()), "tempo_permute_pad")


def tempo_ffn_gate_up(shape, a_q, a_sf, packed, inst_off, m_pad, h_q, h_sf, status):
    _check(_lib.tempo_ffn_gate_up(ctypes.byref(shape), _ptr(a_q, torch.uint8), _ptr(a_sf, torch.uint8),
                                  _ptr(packed, torch.uint8), _ptr(inst_off, torch.int32), _ptr(m_pad, torch.int32),
                                  _ptr(h_q, torch.uint8), _ptr(h_sf, torch.uint8), _ptr(status, torch.int32),
                                  _stream()), "tempo_ffn_gate_up")


def tempo_ffn_down(shape, h_q, h_sf, packed, inst_off, m_pad, y_bf16, status):
    _check(_lib.tempo_ffn_down(ctypes.byref(shape), _ptr(h_q, torch.uint8), _ptr(h_sf, torch.uint8),
                               _ptr(packed, torch.uint8), _ptr(inst_off, torch.int32), _ptr(m_pad, torch.int32),
                               _ptr(y_bf16, torch.bfloat16), _ptr(status, torch.int32), _stream()), "tempo_ffn_down")


def tempo_grouped_ffn(shape, a_q, a_sf, packed, inst_off, m_pad, h_q, h_sf, y_bf16, status, workspace):
    _check(_lib.tempo_grouped_ffn(ctypes.byref(shape), _ptr(a_q, torch.uint8), _ptr(a_sf, torch.uint8),
                                  _ptr(packed, torch.uint8), _ptr(inst_off, torch.int32), _ptr(m_pad, torch.int32),
                                  _ptr(h_q, torch.uint8), _ptr(h_sf, torch.uint8), _ptr(y_bf16, torch.bfloat16),
                                  _ptr(status, torch.int32), _ptr(workspace, torch.uint8), _stream()),
           "tempo_grouped_ffn")


def tempo_token_sf_bytes(shape: TempoShape) -> int:
    out = ctypes.c_size_t(0)
    _check(_lib.tempo_token_sf_bytes(ctypes.byref(shape), ctypes.byref(out)), "tempo_token_sf_bytes")
    return out.value


def tempo_quantize_tokens(shape, x_bf16, n_valid, x_q, x_sf, status):
    _check(_lib.tempo_quantize_tokens(ctypes.byref(shape), _ptr(x_bf16, torch.bfloat16), _ptr(n_valid, torch.int32),
                                      _ptr(x_q, torch.uint8), _ptr(x_sf, torch.uint8), _ptr(status, torch.int32),
                                      _stream()), "tempo_quantize_tokens")


def tempo_grouped_ffn_gather(shape, x_q, x_sf, row_pair, packed, inst_off, m_pad, h_q, h_sf, y_bf16, status, workspace):
    _check(_lib.tempo_grouped_ffn_gather(ctypes.byref(shape), _ptr(x_q, torch.uint8), _ptr(x_sf, torch.uint8),
                                         _ptr(row_pair, torch.int32), _ptr(packed, torch.uint8),
                                         _ptr(inst_off, torch.int32), _ptr(m_pad, torch.int32), _ptr(h_q, torch.uint8),
                                         _ptr(h_sf, torch.uint8), _ptr(y_bf16, torch.bfloat16),
                                         _ptr(status, torch.int32), _ptr(workspace, torch.uint8), _stream()),
           "tempo_grouped_ffn_gather")


def tempo_grouped_ffn_bounded(shape, a_q, a_sf, packed, inst_off, m_pad, h_q, h_sf, y_bf16, status, workspace,
                              wait_limit_ns):
    _check(_lib.tempo_grouped_ffn_bounded(ctypes.byref(shape), _ptr(a_q, torch.uint8), _ptr(a_sf, torch.uint8),
                                          _ptr(packed, torch.uint8), _ptr(inst_off, torch.int32),
                                          _ptr(m_pad, torch.int32), _ptr(h_q, torch.uint8), _ptr(h_sf, torch.uint8),
                                          _ptr(y_bf16, torch.bfloat16), _ptr(status, torch.int32),
                                          _ptr(workspace, torch.uint8), ctypes.c_uint64(int(wait_limit_ns)), _stream()),
           "tempo_grouped_ffn_bounded")


def tempo_grouped_ffn_static(shape, a_q, a_sf, packed, inst_off, m_pad, h_q, h_sf, y_bf16, status):
    """tempo_grouped_ffn for callers that cannot provide scratch memory: the kernel's counters live in an
    array built into the library (M_cap <= 2,097,152 rows).  Nothing is allocated.  Calls on one GPU must
    not overlap; the first call on a device should come before any stream capture."""
    _check(_lib.tempo_grouped_ffn_static(ctypes.byref(shape), _ptr(a_q, torch.uint8), _ptr(a_sf, torch.uint8),
                                         _ptr(packed, torch.uint8), _ptr(inst_off, torch.int32),
                                         _ptr(m_pad, torch.int32), _ptr(h_q, torch.uint8), _ptr(h_sf, torch.uint8),
                                         _ptr(y_bf16, torch.bfloat16), _ptr(status, torch.int32), _stream()),
           "tempo_grouped_ffn_static")


def tempo_unpermute_combine(shape, y_bf16, pair_row, topk_w, n_valid, out_bf16, status):
    _check(_lib.tempo_unpermute_combine(ctypes.byref(shape), _ptr(y_bf16, torch.bfloat16),
                                        _ptr(pair_row, torch.int32), _ptr(topk_w, torch.float32),
                                        _ptr(n_valid, torch.int32), _ptr(out_bf16, torch.bfloat16),
                                        _ptr(status, torch.int32), _stream()), "tempo_unpermute_combine")


def tempo_count_dispatch_masked(shape, max_m, topk_ids, n_valid, replica_map, quota, cum_counts, counts, inst_count,
                                inst_off, pair_row, row_pair, tile_inst, m_pad, status):
    i32 = torch.int32
    _check(_lib.tempo_count_dispatch_masked(ctypes.byref(shape), ctypes.c_int32(max_m), _ptr(topk_ids, i32),
                                            _ptr(n_valid, i32), _ptr(replica_map, i32), _ptr(quota, i32),
                                            _ptr(cum_counts, i32), _ptr(counts, i32), _ptr(inst_count, i32),
                                            _ptr(inst_off, i32), _ptr(pair_row, i32), _ptr(row_pair, i32),
                                            _ptr(tile_inst, i32), _ptr(m_pad, i32), _ptr(status, i32), _stream()),
           "tempo_count_dispatch_masked")


def tempo_permute_pad_masked(shape, x_bf16, row_pair, pair_row, tile_inst, m_pad, a_q, a_sf, status):
    i32 = torch.int32
    _check(_lib.tempo_permute_pad_masked(ctypes.byref(shape), _ptr(x_bf16, torch.bfloat16), _ptr(row_pair, i32),
                                         _ptr(pair_row, i32), _ptr(tile_inst, i32), _ptr(m_pad, i32),
                                         _ptr(a_q, torch.uint8), _ptr(a_sf, torch.uint8), _ptr(status, i32), _stream()),
           "tempo_permute_pad_masked")


def tempo_grouped_ffn_masked(shape, max_m, a_q, a_sf, packed, inst_count, h_q, h_sf, y_bf16, status, workspace):
    _check(_lib.tempo_grouped_ffn_masked(ctypes.byref(shape), ctypes.c_int32(max_m), _ptr(a_q, torch.uint8),
                                         _ptr(a_sf, torch.uint8), _ptr(packed, torch.uint8),
                                         _ptr(inst_count, torch.int32), _ptr(h_q, torch.uint8), _ptr(h_sf, torch.uint8),
                                         _ptr(y_bf16, torch.bfloat16), _ptr(status, torch.int32),
                                         _ptr(workspace, torch.uint8), _stream()), "tempo_grouped_ffn_masked")


def tempo_packed_weight_bytes_bf16(shape: TempoShape) -> int:
    out = ctypes.c_size_t(0)
    _check(_lib.tempo_packed_weight_bytes_bf16(ctypes.byref(shape), ctypes.byref(out)), "tempo_packed_weight_bytes_bf16")
    return out.value


def tempo_pack_weights_bf16(shape, w13_bf16, w2_bf16, packed):
    _check(_lib.tempo_pack_weights_bf16(ctypes.byref(shape), _ptr(w13_bf16, torch.bfloat16), _ptr(w2_bf16, torch.bfloat16),
                                        _ptr(packed, torch.uint8), _stream()), "tempo_pack_weights_bf16")


def tempo_permute_pad_bf16(shape, x_bf16, row_pair, m_pad, a_bf16, status):
    _check(_lib.tempo_permute_pad_bf16(ctypes.byref(shape), _ptr(x_bf16, torch.bfloat16), _ptr(row_pair, torch.int32),
                                       _ptr(m_pad, torch.int32), _ptr(a_bf16, torch.bfloat16), _ptr(status, torch.int32),
                                       _stream()), "tempo_permute_pad_bf16")


def tempo_grouped_ffn_bf16(shape, a_bf16, packed, inst_off, m_pad, h_bf16, y_bf16, status, workspace):
    _check(_lib.tempo_grouped_ffn_bf16(ctypes.byref(shape), _ptr(a_bf16, torch.bfloat16), _ptr(packed, torch.uint8),
                                       _ptr(inst_off, torch.int32), _ptr(m_pad, torch.int32),
                                       _ptr(h_bf16, torch.bfloat16), _ptr(y_bf16, torch.bfloat16),
                                       _ptr(status, torch.int32), _ptr(workspace, torch.uint8), _stream()),
           "tempo_grouped_ffn_bf16")


# ------------------------------------------------------------------------------------------------
# A rank's device buffers: plain allocation and upload, no arithmetic.
# ------------------------------------------------------------------------------------------------

class RankBuffers:
    """Device buffers of one expert-parallel rank for a fixed shape (allocated once, reused per step)."""

    def __init__(self, T, k, E, G_max, R_max, d, f, M_cap=None, device="cuda"):
        dev = torch.device(device)
        probe = make_shape(T, k, E, G_max, R_max, d, f, 128)
        self.M_cap = tempo_m_cap_bound(probe) if M_cap is None else M_cap
        self.shape = make_shape(T, k, E, G_max, R_max, d, f, self.M_cap)
        self.T, self.k, self.E, self.G_max, self.R_max, self.d, self.f = T, k, E, G_max, R_max, d, f
        i32 = dict(dtype=torch.int32, device=dev)
        u8 = dict(dtype=torch.uint8, device=dev)
        self.topk_ids = torch.zeros(T, k, **i32)
        self.topk_w = torch.zeros(T, k, dtype=torch.float32, device=dev)
        self.n_valid = torch.full((1,), T, **i32)
        self.replica_map = torch.full((E, R_max), -1, **i32)
        self.quota = torch.zeros(E, R_max, **i32)
        self.x = torch.zeros(T, d, dtype=torch.bfloat16, device=dev)
        self.cum_counts = torch.zeros(E, **i32)           # u32 counter kept in an int32 tensor
        self.counts = torch.zeros(E, **i32)
        self.inst_count = torch.zeros(G_max, **i32)
        self.inst_off = torch.zeros(G_max + 1, **i32)
        self.pair_row = torch.full((T * k,), -1, **i32)
        self.row_pair = torch.full((self.M_cap,), -1, **i32)
        self.tile_inst = torch.full((self.M_cap // 128,), -1, **i32)
        self.m_pad = torch.zeros(1, **i32)
        self.status = torch.zeros(1, **i32)
        self.a_q = torch.zeros(self.M_cap, d, **u8)
        self.a_sf = torch.full((tempo_sf_bytes(self.M_cap, d),), 127, **u8)
        self.h_q = torch.zeros(self.M_cap, f, **u8)
        self.h_sf = torch.full((tempo_sf_bytes(self.M_cap, f),), 127, **u8)
        self.y = torch.zeros(self.M_cap, d, dtype=torch.bfloat16, device=dev)
        self.out = torch.zeros(T, d, dtype=torch.bfloat16, device=dev)
        self.workspace = torch.zeros(tempo_workspace_bytes(self.shape), **u8)   # counters start at zero
        self.x_q = torch.zeros(T, d, **u8)                  # per-token quantised activations (gather form)
        self.x_sf = torch.full((tempo_token_sf_bytes(self.shape),), 127, **u8)
        self.packed = None

    def pack_weights(self, w13_q, w13_s, w2_q, w2_s):
        """Upload canonical per-slot weights (host or device tensors) and re-lay them once."""
        dev = self.x.device
        self.packed = torch.empty(tempo_packed_weight_bytes(self.shape), dtype=torch.uint8, device=dev)
        args = [torch.as_tensor(a).to(dev).contiguous() for a in (w13_q, w13_s, w2_q, w2_s)]
        tempo_pack_weights(self.shape, *args, self.packed, self.status)
        torch.cuda.synchronize()
        return self.packed

    def run_block(self, packed=None):
        """One pass of the whole hot path: the four C-ABI steps, enqueued back to back."""
        s = self.shape
        packed = self.packed if packed is None else packed
        tempo_count_dispatch(s, self.topk_ids, self.n_valid, self.replica_map, self.quota, self.cum_counts,
                             self.counts, self.inst_count, self.inst_off, self.pair_row, self.row_pair,
                             self.tile_inst, self.m_pad, self.status)
        tempo_permute_pad(s, self.x, self.row_pair, self.m_pad, self.a_q, self.a_sf, self.status, pair_row=self.pair_row)
        tempo_grouped_ffn(s, self.a_q, self.a_sf, packed, self.inst_off, self.m_pad, self.h_q, self.h_sf, self.y,
                          self.status, self.workspace)
        tempo_unpermute_combine(s, self.y, self.pair_row, self.topk_w, self.n_valid, self.out, self.status)

    def run_block_gather(self, packed=None):
        """The same block with the gather fused into the FFN: quantise tokens (beside the dispatch), then the
        FFN fetches its rows by row_pair.  Same results bit for bit; a_q / a_sf are not written."""
        s = self.shape
        packed = self.packed if packed is None else packed
        tempo_count_dispatch(s, self.topk_ids, self.n_valid, self.replica_map, self.quota, self.cum_counts,
                             self.counts, self.inst_count, self.inst_off, self.pair_row, self.row_pair,
                             self.tile_inst, self.m_pad, self.status)
        tempo_quantize_tokens(s, self.x, self.n_valid, self.x_q, self.x_sf, self.status)
        tempo_grouped_ffn_gather(s, self.x_q, self.x_sf, self.row_pair, packed, self.inst_off, self.m_pad, self.h_q,
                                 self.h_sf, self.y, self.status, self.workspace)
        tempo_unpermute_combine(s, self.y, self.pair_row, self.topk_w, self.n_valid, self.out, self.status)

    def run_block_masked(self, max_m, packed=None):
        """One pass of the block in the masked layout (instance i at rows [i*max_m, (i+1)*max_m))."""
        s = self.shape
        packed = self.packed if packed is None else packed
        tempo_count_dispatch_masked(s, max_m, self.topk_ids, self.n_valid, self.replica_map, self.quota, self.cum_counts,
                                    self.counts, self.inst_count, self.inst_off, self.pair_row, self.row_pair,
                                    self.tile_inst, self.m_pad, self.status)
        tempo_permute_pad_masked(s, self.x, self.row_pair, self.pair_row, self.tile_inst, self.m_pad, self.a_q, self.a_sf,
                                 self.status)
        tempo_grouped_ffn_masked(s, max_m, self.a_q, self.a_sf, packed, self.inst_count, self.h_q, self.h_sf, self.y,
                                 self.status, self.workspace)
        tempo_unpermute_combine(s, self.y, self.pair_row, self.topk_w, self.n_valid, self.out, self.status)

    # ---- bf16 variant (separate activation / weight buffers, allocated on first use) ----
    def pack_weights_bf16(self, w13, w2):
        dev = self.x.device
        self.packed_bf16 = torch.empty(tempo_packed_weight_bytes_bf16(self.shape), dtype=torch.uint8, device=dev)
        a = torch.as_tensor(w13).to(dev).to(torch.bfloat16).contiguous()
        b = torch.as_tensor(w2).to(dev).to(torch.bfloat16).contiguous()
        tempo_pack_weights_bf16(self.shape, a, b, self.packed_bf16)
        torch.cuda.synchronize()
        self.alloc_bf16()
        return self.packed_bf16

    def alloc_bf16(self):
        dev_kw = dict(dtype=torch.bfloat16, device=self.x.device)
        self.a_bf16 = torch.zeros(self.M_cap, self.d, **dev_kw)
        self.h_bf16 = torch.zeros(self.M_cap, self.f, **dev_kw)

    def run_block_bf16(self, packed=None):
        """One pass of the block with the bf16 steps 2 and 3."""
        s = self.shape
        packed = self.packed_bf16 if packed is None else packed
        tempo_count_dispatch(s, self.topk_ids, self.n_valid, self.replica_map, self.quota, self.cum_counts,
                             self.counts, self.inst_count, self.inst_off, self.pair_row, self.row_pair,
                             self.tile_inst, self.m_pad, self.status)
        tempo_permute_pad_bf16(s, self.x, self.row_pair, self.m_pad, self.a_bf16, self.status)
        tempo_grouped_ffn_bf16(s, self.a_bf16, packed, self.inst_off, self.m_pad, self.h_bf16, self.y, self.status,
                               self.workspace)
        tempo_unpermute_combine(s, self.y, self.pair_row, self.topk_w, self.n_valid, self.out, self.status)

    def upload(self, wl, with_weights=True):
        """Copy a seeded workload (workloads.Workload) into the device buffers."""
        dev = self.x.device
        self.topk_ids.copy_(torch.from_numpy(wl.topk_ids))
        self.topk_w.copy_(torch.from_numpy(wl.topk_w))
        self.n_valid.fill_(int(wl.n_valid))
        self.replica_map.copy_(torch.from_numpy(wl.replica_map))
        self.quota.copy_(torch.from_numpy(wl.quota))
        if wl.x is not None:
            self.x.copy_(torch.from_numpy(wl.x).to(torch.bfloat16))
        if with_weights:
            self.pack_weights(*wl.slot_weights())
        torch.cuda.synchronize()
        return self

    @classmethod
    def for_workload(cls, wl, M_cap=None, device="cuda", with_weights=True):
        buf = cls(wl.T, wl.k, wl.E, wl.G_max, wl.R_max, wl.d, wl.f, M_cap=M_cap, device=device)
        return buf.upload(wl, with_weights=with_weights)
