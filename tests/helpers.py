"""Small host-side helpers shared by the tests (no method arithmetic of the library or the oracle)."""
import numpy as np
import torch


def to_bf16_bits(x) -> np.ndarray:
    """Round a float array to bf16 (nearest-even, torch) and return the raw bits as uint16."""
    t = torch.as_tensor(np.asarray(x, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16).copy()


def from_bf16_bits(bits) -> np.ndarray:
    """Exact widening of bf16 bits to float64."""
    b = np.ascontiguousarray(bits, dtype=np.uint16)
    return (b.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def bf16_round(x) -> np.ndarray:
    return from_bf16_bits(to_bf16_bits(x))


def identity_layout(page_counts, S, ctx=None):
    """page_base / ctx_len for requests laid out back to back with full pages."""
    page_counts = np.asarray(page_counts, dtype=np.int64)
    page_base = np.concatenate([[0], np.cumsum(page_counts)]).astype(np.int64)
    ctx_len = ctx
    if ctx_len is None:
        ctx_len = (page_counts * S).astype(np.int32)
    return page_base, np.asarray(ctx_len, dtype=np.int32)
