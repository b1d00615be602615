"""Helpers for the GPU parity tests: canary-padded device buffers and oracle comparison."""
import numpy as np
import torch

import paper_2504_20634_b200 as fbsr
from oracle import capi

CANARY = 0xA5
PAD = 64          # bytes of guard before and after every output buffer


def guarded(n, dtype, device="cuda", misalign=0):
    """A device tensor of n elements whose storage is surrounded by canary bytes.
    misalign: extra elements to skip so that the view starts off a 16-byte boundary."""
    item = torch.empty(0, dtype=dtype).element_size()
    raw = torch.full((2 * PAD + (n + misalign) * item,), CANARY, dtype=torch.uint8, device=device)
    view = raw[PAD + misalign * item: PAD + (misalign + n) * item].view(dtype)
    return raw, view


def canaries_intact(raw, n, dtype, misalign=0):
    item = torch.empty(0, dtype=dtype).element_size()
    head = raw[: PAD + misalign * item]
    tail = raw[PAD + (misalign + n) * item:]
    return bool((head == CANARY).all()) and bool((tail == CANARY).all())


def to_np(t):
    if t.dtype == torch.uint16:
        return t.view(torch.int16).cpu().numpy().view(np.uint16)
    if t.dtype == torch.uint32:
        return t.view(torch.int32).cpu().numpy().view(np.uint32)
    return t.cpu().numpy()


def from_np_u32(a, device="cuda"):
    return torch.from_numpy(a.view(np.int32).copy()).to(device).view(torch.uint32)


def from_np_codes(a, device="cuda"):
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16).copy()).to(device).view(torch.uint16)
    return torch.from_numpy(a.copy()).to(device)


def mixed_inputs(n, seed, fmt):
    """Random binary32 patterns covering the target's normal, subnormal, underflow and overflow
    ranges, with every special value sprinkled in."""
    from helpers import random_f32, edge_values_f32
    rng = np.random.default_rng(seed)
    lo, hi = {"bf16": (-126, 127), "fp16": (-30, 17), "e4m3": (-14, 10), "e5m2": (-22, 17), "b8p4": (-15, 9)}[fmt]
    pats = random_f32(rng, n, lo, hi)
    edges = edge_values_f32()
    if n >= 4 * edges.size:
        pos = rng.choice(n, size=edges.size, replace=False)
        pats[pos] = edges
        sub = rng.choice(n, size=min(16, n // 8), replace=False)
        pats[sub] = rng.integers(0, 1 << 23, size=sub.size, dtype=np.uint32)      # binary32 subnormals
    return pats.view(np.float32)


def assert_codes_equal(got_t, expect_np, what=""):
    got = to_np(got_t)
    if not np.array_equal(got, expect_np):
        bad = np.nonzero(got != expect_np)[0]
        raise AssertionError("%s: %d of %d codes differ, first at %d: got %#x expect %#x"
                             % (what, bad.size, got.size, bad[0], got[bad[0]], expect_np[bad[0]]))
