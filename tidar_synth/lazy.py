"""Weight containers that hand a big model to a float64 consumer piece by piece.

No arithmetic of the method lives here: only "give me layer l as float64 arrays" and "upcast
the rows / the chunk of this bf16 matrix that is being read".  A consumer that iterates over
``layers`` once per pass (the CPU oracle does) then never holds more than one layer in
float64, so an 8B-class model fits an ordinary host.
"""
from __future__ import annotations

import time

import numpy as np
import torch

from .generators import ModelShape, gen_model_weights

_PRODUCTION = [0.0]


def production_seconds() -> float:
    """Wall time this module has spent so far producing float64 pieces (generation, copies to the
    host, upcasts): a caller that times its own arithmetic around lazy weights subtracts the growth."""
    return _PRODUCTION[0]


class LazyLayers:
    """Iterable over the layers of ``shape``: layer l's weights are generated (on ``device``, from
    the same counter-based generator as every other copy of the model) and upcast to float64 when
    the loop reaches l, and dropped afterwards."""

    def __init__(self, shape: ModelShape, device="cpu"):
        self.shape, self.device = shape, device

    def __len__(self):
        return self.shape.n_layers

    def __iter__(self):
        for l in range(self.shape.n_layers):
            t0 = time.perf_counter()
            lay = gen_model_weights(self.shape, device=self.device, layers=[l], with_head=False)["layers"][0]
            out = {k: (v if k == "index" else v.float().cpu().numpy().astype(np.float64)) for k, v in lay.items()}
            del lay
            _PRODUCTION[0] += time.perf_counter() - t0
            yield out


class LazyRows:
    """A [rows, d] bf16 matrix kept as it is and upcast to float64 only where it is read:
    ``m[ids]`` (some rows) and ``y @ m.T`` (all of it, in chunks of rows)."""
    __array_ufunc__ = None          # makes ``ndarray @ self`` call __rmatmul__ instead of converting self

    def __init__(self, tensor: torch.Tensor, transposed: bool = False):
        self.t, self.transposed = tensor, transposed

    def _f64(self, t):
        t0 = time.perf_counter()
        a = t.float().cpu().numpy().astype(np.float64)
        _PRODUCTION[0] += time.perf_counter() - t0
        return a

    def __getitem__(self, ids):
        idx = torch.as_tensor(np.asarray(ids), device=self.t.device)
        return self._f64(self.t[idx])

    @property
    def T(self):
        return LazyRows(self.t, not self.transposed)

    def __rmatmul__(self, y):
        assert self.transposed, "only y @ m.T is supported"
        out = np.empty((y.shape[0], self.t.shape[0]), dtype=np.float64)
        for v0 in range(0, self.t.shape[0], 16384):
            out[:, v0:v0 + 16384] = y @ self._f64(self.t[v0:v0 + 16384]).T
        return out


def lazy_model_weights(shape: ModelShape, device="cpu") -> dict:
    """A weight dict in the generator's layout whose big parts are lazy: ``embed`` / ``lm_head`` are
    :class:`LazyRows`, ``layers`` is a :class:`LazyLayers`, ``final_norm`` a float64 array."""
    head = gen_model_weights(shape, device=device, layers=[])
    w = {"embed": LazyRows(head["embed"]), "final_norm": head["final_norm"].float().cpu().numpy().astype(np.float64)}
    w["lm_head"] = w["embed"] if shape.tie_lm_head else LazyRows(head["lm_head"])
    w["layers"] = LazyLayers(shape, device)
    return w
