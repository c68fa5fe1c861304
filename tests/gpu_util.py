"""Helpers of the GPU parity tests: decode library layouts on the host (index formulas from tempo.h)."""
import numpy as np
import torch


def sf_decode(sf_bytes: np.ndarray, rows: int, cols: int) -> np.ndarray:
    """Scale bytes in 512-byte atoms -> f32 scales [rows, cols/128] (2^(b-127))."""
    kb_n = cols // 128
    J = (kb_n + 3) // 4
    r = np.arange(rows)[:, None]
    kb = np.arange(kb_n)[None, :]
    idx = ((r // 128) * J + kb // 4) * 512 + (r % 32) * 16 + ((r % 128) // 32) * 4 + kb % 4
    b = sf_bytes[idx].astype(np.int32)
    return np.exp2((b - 127).astype(np.float64)).astype(np.float32)


def codes_equal_mod_signed_zero(a: np.ndarray, b: np.ndarray) -> np.ndarray:
    za = (a & 0x7F) == 0
    zb = (b & 0x7F) == 0
    return (a == b) | (za & zb)


def to_np(t: torch.Tensor) -> np.ndarray:
    if t.dtype == torch.bfloat16:
        return t.float().cpu().numpy()
    return t.cpu().numpy()


def dispatch_outputs(buf):
    return dict(counts=to_np(buf.counts), inst_count=to_np(buf.inst_count), inst_off=to_np(buf.inst_off),
                pair_row=to_np(buf.pair_row), row_pair=to_np(buf.row_pair), tile_inst=to_np(buf.tile_inst),
                m_pad=int(buf.m_pad.item()), status=int(buf.status.item()) & 0xFFFFFFFF,
                cum_counts=to_np(buf.cum_counts).view(np.uint32))
