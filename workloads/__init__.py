"""Seeded synthetic inputs for the VADUSA tree draft-and-verify step.

This package only *makes inputs*: model shapes, random-init weights, phoneme and
prompt token streams, static candidate-tree templates, random tree topologies,
KV block tables.  It contains none of the method's arithmetic (no transformer
forward, no sampling, no acceptance rule), so both the CPU oracle's tests and
the CUDA path's harness may import it without sharing any code of the method.
"""
from .configs import ModelShape, Workload, WORKLOADS, workload, toy_workload
from .weights import make_weights, round_to_bf16_values
from .streams import phonemes, markov_prompt, prefix_for, ragged_lengths
from .trees import (static_template, random_topology, chain_template,
                    ancestor_masks, depths_of, validate_template, TreeTemplate)
from .paging import shuffled_block_table

__all__ = [
    "ModelShape", "Workload", "WORKLOADS", "workload", "toy_workload",
    "make_weights", "round_to_bf16_values",
    "phonemes", "markov_prompt", "prefix_for", "ragged_lengths",
    "static_template", "random_topology", "chain_template", "ancestor_masks",
    "depths_of", "validate_template", "TreeTemplate", "shuffled_block_table",
]
