"""Seeded synthetic inputs for the recursive-dataflow workloads.

This package only *draws* inputs (integers, tree shapes, token ids, labels,
parameter tensors).  It contains none of the method's arithmetic: no tag
handling, no cell evaluation, no gradients.  Both the CPU oracle and the CUDA
path are fed from here so that they see identical arrays.
"""
from .gen import (  # noqa: F401
    DEFAULT_SEED,
    TreeBatch,
    bf16_round,
    chain_tree_shape,
    config,
    fib_batch,
    perfect_tree_shape,
    random_split_shape,
    subset_trees,
    topdown_batch,
    topdown_params,
    tree_batch_from_shapes,
    treelstm_params,
    treernn_params,
)
