"""Python binding of the host-side archive of kernel variants (``include/kf_archive.h``): argument
marshalling only, the bookkeeping itself runs in the kf library.

The paper files its candidate kernels in a MAP-Elites grid over (d_mem, d_algo, d_sync), records
parent -> child transitions and derives gradient estimates from them (Sections 3.2 and 3.3); the
parameter sweep of this package uses the same structures to file the variants it times.
"""
from __future__ import annotations

import ctypes
from typing import Optional, Sequence

from . import binding

IMPROVEMENT, NEUTRAL, REGRESSION = 1, 0, -1
_BAD_ARG = -100
_I3 = ctypes.c_int32 * 3
_ready = False


def _lib():
    global _ready
    L = binding.lib()
    if not _ready:
        vp, i32, i64, dbl = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_double
        L.kf_fitness.argtypes = [i32, i32, dbl, dbl]
        L.kf_fitness.restype = dbl
        L.kf_archive_create.argtypes = [i32, dbl, dbl]
        L.kf_archive_create.restype = vp
        L.kf_archive_destroy.argtypes = [vp]
        L.kf_archive_destroy.restype = None
        L.kf_archive_insert.argtypes = [vp, ctypes.POINTER(i32), dbl, i64, ctypes.POINTER(i32), dbl, i64]
        L.kf_archive_insert.restype = i32
        L.kf_archive_cell.argtypes = [vp, ctypes.POINTER(i32), ctypes.POINTER(dbl), ctypes.POINTER(i64)]
        L.kf_archive_cell.restype = i32
        L.kf_archive_transitions.argtypes = [vp]
        L.kf_archive_transitions.restype = i32
        L.kf_archive_gradient.argtypes = [vp, ctypes.POINTER(i32), i64, ctypes.POINTER(dbl), ctypes.POINTER(dbl)]
        L.kf_archive_gradient.restype = i32
        L.kf_archive_sampling_weights.argtypes = [vp, i64, ctypes.POINTER(i32), ctypes.POINTER(dbl)]
        L.kf_archive_sampling_weights.restype = i32
        _ready = True
    return L


def fitness(compiled: bool, correct: bool, speedup: float, target: float = 2.0) -> float:
    """f(k) of Section 3.2: 0 / 0.1 / 0.5 + 0.5 min(1, speedup / target)."""
    return float(_lib().kf_fitness(int(bool(compiled)), int(bool(correct)), float(speedup), float(target)))


class Archive:
    """One elite per cell of the 4 x 4 x 4 grid, a ring buffer of transitions, gradient estimates."""

    def __init__(self, capacity: int = 256, half_life: float = 50.0, low_quality: float = 0.5):
        self._L = _lib()
        self._h = self._L.kf_archive_create(int(capacity), float(half_life), float(low_quality))
        if not self._h:
            raise ValueError("kf_archive_create rejected its arguments")

    def close(self):
        if self._h:
            self._L.kf_archive_destroy(self._h)
            self._h = None

    def __del__(self):
        self.close()

    def insert(self, coords: Sequence[int], fit: float, ident: int = 0, parent: Optional[Sequence[int]] = None,
               parent_fit: float = 0.0, iteration: int = 0) -> int:
        r = self._L.kf_archive_insert(self._h, _I3(*coords), float(fit), int(ident),
                                      _I3(*parent) if parent is not None else None, float(parent_fit), int(iteration))
        if r == _BAD_ARG:
            raise ValueError(f"coordinates outside the grid: {coords} / {parent}")
        return r

    def cell(self, coords: Sequence[int]):
        f, i = ctypes.c_double(0.0), ctypes.c_int64(0)
        r = self._L.kf_archive_cell(self._h, _I3(*coords), ctypes.byref(f), ctypes.byref(i))
        if r == _BAD_ARG:
            raise ValueError(f"coordinates outside the grid: {coords}")
        return (f.value, i.value) if r == 1 else None

    def transitions(self) -> int:
        return int(self._L.kf_archive_transitions(self._h))

    def gradient(self, coords: Sequence[int], now: int):
        """(combined[3], F[3], R[3], E[3]) for one cell (Section 3.3, Eq. 1-3, weights 0.4 / 0.4 / 0.2)."""
        g, comp = (ctypes.c_double * 3)(), (ctypes.c_double * 9)()
        if self._L.kf_archive_gradient(self._h, _I3(*coords), int(now), g, comp) != 0:
            raise ValueError(f"coordinates outside the grid: {coords}")
        return list(g), list(comp[0:3]), list(comp[3:6]), list(comp[6:9])

    def sampling_weights(self, now: int) -> dict:
        """Occupied cell -> selection probability, proportional to exp(|gradient|_2)."""
        c, w = (ctypes.c_int32 * 192)(), (ctypes.c_double * 64)()
        n = self._L.kf_archive_sampling_weights(self._h, int(now), c, w)
        return {(c[3 * i], c[3 * i + 1], c[3 * i + 2]): w[i] for i in range(n)}
