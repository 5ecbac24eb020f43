"""Seeded synthetic inputs for the PipeMare hot path.

This package serves both the CPU oracle and the CUDA library's tests and
benchmark.  It holds workload descriptions (shapes, delays, hyper-parameters),
a counter-based random number generator, and the recipes that turn seeds into
initial weights, input batches and targets.  It contains none of the method's
arithmetic: no delayed update, no learning-rate rescheduling, no discrepancy
correction, no backward pass.
"""
from .rng import uniform01, normal, randint, zipf_ranks  # noqa: F401
from .configs import (  # noqa: F401
    Workload, LinearSpec, pipemare_delays, mlp_workload, cfg1, cfg3, cfg3_small,
    update_sweep_case, init_stage_params, teacher_params, batch, round_to_bf16,
    StageSpec, encoder_workload, cfg4, cfg4_small, init_encoder_params, token_batch,
    encdec_workload, cfg5, cfg5_cut, cfg5_small, seq2seq_batch, stochastic_delays,
)
