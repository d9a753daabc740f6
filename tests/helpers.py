"""Shared test plumbing: build one seeded workload and present it to both sides.

The oracle receives float64 arrays holding the exact storage-precision values;
the CUDA path receives the raw bf16 bit patterns / fp32 arrays. No arithmetic of
the method lives here.
"""

from __future__ import annotations

from dataclasses import replace

import numpy as np

from paper_2609_36222_b200 import workloads as wl


class HostLayer:
    """All tensors of one layer on the host, with lazy per-expert decoding for the oracle."""

    def __init__(self, cfg, seed=0, layer=0, T=None, experts="all", planted_alpha=None, bias_scale=1.0):
        self.cfg = cfg
        self.seed, self.layer = seed, layer
        self.T = cfg.T if T is None else T
        self.hidden_bits = wl.hidden_bits(cfg, self.T, seed, layer)
        self.small = wl.small_tensors(cfg, seed, layer)
        if bias_scale != 1.0:
            self.small["router_bias"] = wl.router_bias(cfg, seed, layer, bias_scale)
        self._bits = None
        self._cache = {}
        if experts == "all":
            self._bits = wl.expert_weights_host_all(cfg, seed, layer)
            if planted_alpha is not None:
                self._bits["w_gate"] = wl.plant_energy_direction(cfg, self._bits["w_gate"], planted_alpha, seed)

    # -- oracle-side views (float64, exact values)
    @property
    def z(self):
        return wl.bf16_bits_to_f64(self.hidden_bits)

    @property
    def router_w(self):
        return wl.bf16_bits_to_f64(self.small["router_w"])

    @property
    def router_bias(self):
        return self.small["router_bias"].astype(np.float64)

    @property
    def pred_A(self):
        return wl.bf16_bits_to_f64(self.small["pred_A"])

    @property
    def pred_b(self):
        return self.small["pred_b"].astype(np.float64)

    def expert_bits(self, u):
        if self._bits is not None:
            return {k: v[u] for k, v in self._bits.items()}
        return wl.expert_weights_host(self.cfg, u, self.seed, self.layer)

    def expert_weights(self, u):
        """(w_gate, w_up, w_down) of expert u as float64 (cached for small layers)."""
        if u in self._cache:
            return self._cache[u]
        b = self.expert_bits(u)
        w = tuple(wl.bf16_bits_to_f64(b[k]) for k in ("w_gate", "w_up", "w_down"))
        if self.cfg.expert_bytes <= (16 << 20):
            self._cache[u] = w
        return w

    def all_bits(self):
        assert self._bits is not None
        return self._bits


def small_cfg(name="unit", d=32, E=8, K=2, I=16, T=5, budgets=(3,)):
    return wl.LayerConfig(name, d=d, E=E, K=K, I=I, T=T, budgets=budgets)


def with_T(cfg, T):
    return replace(cfg, T=T)
