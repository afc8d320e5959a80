"""Seeded synthetic inputs (weights, prompts) shared by the oracle's tests and
the CUDA library's tests and benchmark.  Holds none of the method's arithmetic."""
from .models import (ModelShape, Workload, WORKLOADS, TINY, S1B, S7B, S13B,
                     tensor_shapes, make_weights, make_prompts)
from .prompts import markov_prompt, periodic_prompt
from .orbit import (ScriptedOrbitModel, make_orbit_weights, orbit_continuation, orbit_fork_prompt, orbit_permutation, orbit_prompt,
                    workload_inputs)
from . import rng

__all__ = ["ModelShape", "Workload", "WORKLOADS", "TINY", "S1B", "S7B", "S13B",
           "tensor_shapes", "make_weights", "make_prompts", "markov_prompt",
           "periodic_prompt", "rng", "ScriptedOrbitModel", "make_orbit_weights", "orbit_continuation",
           "orbit_fork_prompt", "orbit_permutation", "orbit_prompt", "workload_inputs"]
