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


# ---------------------------------------------------------------------------- whole tensors through the oracle
class WholeTensorChecker:
    """Runs the scalar oracle over every element of large tensors on all host cores.

    The tensor is cut into pieces of `piece` elements; a pool of threads (ctypes releases the GIL while the C
    oracle runs) calls `fn(a, b)` for every piece [a, b) and collects the first mismatch it reports.  Every
    piece is checked unless the time budget (seconds, over the life of the checker) would be overrun at the
    rate seen so far; then, and only then, later calls check every `stride`-th piece, and what fraction of the
    pieces ran is kept in `self.fraction` and printed, never hidden.
    """

    def __init__(self, budget_s, piece=1 << 20, threads=None):
        import concurrent.futures
        import os
        import time
        self.time = time
        self.threads = threads or max(1, min(64, os.cpu_count() or 1))
        self.pool = concurrent.futures.ThreadPoolExecutor(self.threads)
        self.piece, self.budget = piece, float(budget_s)
        self.spent, self.pieces_run, self.pieces_all = 0.0, 0, 0

    def run(self, n, fn, remaining_calls=1):
        """fn(a, b) -> None or a message.  remaining_calls: how many calls of this size are still to come
        (this one included), used to spread what is left of the budget."""
        starts = list(range(0, n, self.piece))
        stride = 1
        if self.pieces_run:
            per_piece = self.spent / self.pieces_run
            allowed = max(self.budget - self.spent, 0.0) / max(remaining_calls, 1)
            if per_piece * len(starts) > allowed:
                stride = int(per_piece * len(starts) / max(allowed, 1e-9)) + 1
        chosen = starts[::stride]
        if starts and chosen[-1] != starts[-1]:
            chosen.append(starts[-1])                    # the ragged end is always checked
        t0 = self.time.perf_counter()
        for msg in self.pool.map(lambda a: fn(a, min(a + self.piece, n)), chosen):
            if msg is not None:
                raise AssertionError(msg)
        self.spent += self.time.perf_counter() - t0
        self.pieces_run += len(chosen)
        self.pieces_all += len(starts)

    @property
    def fraction(self):
        return self.pieces_run / self.pieces_all if self.pieces_all else 1.0

    def report(self, what):
        line = "%s: oracle checked %d of %d pieces of %d elements (%.1f %%) in %.1f s on %d threads" % (
            what, self.pieces_run, self.pieces_all, self.piece, 100.0 * self.fraction, self.spent, self.threads)
        print(line)
        if self.fraction < 1.0:
            import warnings
            warnings.warn(line + " -- the time budget of %.0f s cut the rest" % self.budget)
        self.pool.shutdown()
        return line


def first_difference(got, expect, base, what):
    """None if equal, else a message naming the first differing element (global index base + i)."""
    if np.array_equal(got, expect):
        return None
    bad = np.nonzero(got != expect)[0]
    return "%s: %d of %d differ, first at element %d: got %#x expect %#x" % (
        what, bad.size, got.size, base + int(bad[0]), int(got[bad[0]]), int(expect[bad[0]]))


def pinned_like(t):
    """A pinned host tensor of the same shape and dtype, with its numpy view (uint16 viewed through int16)."""
    h = torch.empty(t.shape, dtype=t.dtype).pin_memory()
    if t.dtype == torch.uint16:
        return h, h.view(torch.int16).numpy().view(np.uint16)
    if t.dtype == torch.uint32:
        return h, h.view(torch.int32).numpy().view(np.uint32)
    return h, h.numpy()
