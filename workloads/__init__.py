"""Declarative workload descriptions and seeded synthetic-input generators.

Nothing in this package performs any of the method's arithmetic (no training
step, no selection, no perturbation, no counter-based random stream): it only
describes populations (shapes, priors, intervals) and draws the data pools and
initial hyperparameters that both the CPU oracle and the GPU library consume
as inputs.
"""
from .configs import PBTConfig, CONFIGS, get_config  # noqa: F401
from .generate import make_inputs, Inputs  # noqa: F401
