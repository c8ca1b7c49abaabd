"""Canary words around the harness's device allocations.

``GuardedTorch`` stands in for the ``torch`` module inside the binding and the parity harness:
every device tensor they allocate sits between two guard regions filled with a known byte, and
``check`` verifies after a test that no kernel wrote outside the tensor it was given.  Together
with the bounds-checked library (``A2SF_LIBRARY=debug``) this replaces a memory checker.
"""
from __future__ import annotations

import math

GUARD_BYTES = 4096
GUARD_BYTE = 0xA5


class GuardedTorch:
    def __init__(self, real):
        self._real = real
        self._bases = []          # (base uint8 tensor, payload bytes): kept alive until release()
        self.regions_checked = 0

    def __getattr__(self, name):
        return getattr(self._real, name)

    # ---- allocation ------------------------------------------------------------------------
    def _is_device(self, device, pin_memory=False):
        if pin_memory or device is None:
            return False
        return self._real.device(device).type == "cuda"

    def _payload(self, nbytes, device):
        real = self._real
        padded = (nbytes + 255) // 256 * 256
        base = real.empty((GUARD_BYTES + padded + GUARD_BYTES,), dtype=real.uint8, device=device)
        base[:GUARD_BYTES] = GUARD_BYTE
        base[GUARD_BYTES + nbytes:] = GUARD_BYTE          # the padding belongs to the guard
        self._bases.append((base, nbytes))
        return base[GUARD_BYTES:GUARD_BYTES + nbytes]

    def empty(self, *size, dtype=None, device=None, pin_memory=False, **kw):
        if not self._is_device(device, pin_memory):
            return self._real.empty(*size, dtype=dtype, device=device, pin_memory=pin_memory, **kw)
        shape = tuple(size[0]) if len(size) == 1 and not isinstance(size[0], int) else tuple(size)
        dtype = dtype or self._real.float32
        item = self._real.empty((), dtype=dtype).element_size()
        n = math.prod(shape)
        if n == 0:
            return self._real.empty(shape, dtype=dtype, device=device)
        return self._payload(n * item, device).view(dtype).view(shape)

    def empty_strided(self, size, stride, dtype=None, device=None, **kw):
        if not self._is_device(device):
            return self._real.empty_strided(size, stride, dtype=dtype, device=device, **kw)
        dtype = dtype or self._real.float32
        item = self._real.empty((), dtype=dtype).element_size()
        if math.prod(size) == 0:
            return self._real.empty_strided(size, stride, dtype=dtype, device=device)
        extent = 1 + sum((s - 1) * st for s, st in zip(size, stride))
        flat = self._payload(extent * item, device).view(dtype)
        return self._real.as_strided(flat, tuple(size), tuple(stride))

    def empty_like(self, t, **kw):
        if kw or not t.is_cuda:
            return self._real.empty_like(t, **kw)
        return self.empty_strided(tuple(t.shape), tuple(t.stride()), dtype=t.dtype, device=t.device)

    # ---- verification ----------------------------------------------------------------------
    def check(self, what=""):
        """Every guard region of every allocation made so far still holds the guard byte."""
        real = self._real
        for base, nbytes in self._bases:
            lo = base[:GUARD_BYTES]
            hi = base[GUARD_BYTES + nbytes:]
            ok = bool((lo == GUARD_BYTE).all().item()) and bool((hi == GUARD_BYTE).all().item())
            if not ok:
                bad_lo = int((lo != GUARD_BYTE).sum().item())
                bad_hi = int((hi != GUARD_BYTE).sum().item())
                raise AssertionError(f"{what}: a kernel wrote outside a {nbytes}-byte buffer: {bad_lo} guard bytes "
                                     f"changed before it, {bad_hi} after it")
            self.regions_checked += 2
        real.cuda.synchronize()

    def release(self):
        self._bases.clear()
