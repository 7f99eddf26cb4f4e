"""Seeded synthetic inputs (model shapes, weights, request streams).

This package holds none of the serving method's arithmetic: it only draws
random numbers and lays them out.  Both the CPU oracle's tests and the CUDA
path's tests/bench feed from it, so the two see identical inputs.
"""
from .configs import ModelCfg, SchedCfg, CONFIGS, model_cfg, sched_cfg  # noqa: F401
from .weights import weight_layout, make_weights, weights_as_numpy  # noqa: F401
from .workload import make_requests, Request  # noqa: F401
