"""Seeded synthetic inputs shaped like the paper's workloads.

This package only draws inputs (weights, bases, activations).  It holds none of
the method's arithmetic and is imported by the tests and by ``bench.py``; the
CUDA package and the oracle do not depend on it.
"""
from .generators import (  # noqa: F401
    seed_for, gen_weight, gen_basis, gen_true_basis, gen_activations,
    to_bf16_bits, bits_of, store_basis,
)
from .configs import (  # noqa: F401
    GroupSpec, StackSpec, config1, config1_fast, config2, config3, config4, config5,
    materialize_group, gptj_groups, opt_groups, gpt2_groups,
)
