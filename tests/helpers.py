"""Shared test helpers: cached host weights and oracle construction."""
import numpy as np

from workloads.generate import WeightStore


class HostWeights:
    """name -> float array, converted once; individual tensors can be overridden."""

    def __init__(self, store: WeightStore, dtype=np.float64):
        self.store, self.dtype, self.cache = store, dtype, {}

    def __call__(self, name):
        if name not in self.cache:
            self.cache[name] = self.store.host(name, self.dtype)
        return self.cache[name]

    def override(self, name, value):
        self.cache[name] = np.asarray(value, dtype=self.dtype)
        return self
