"""Recursive function definitions as one static tagged dataflow graph, executed
on a B200 (sm_100a): tag-push / tag-pop (Call_i / Return_i), (node, tag)
matching and wave-batched firing in hand-written CUDA behind a C boundary
(include/rdf.h).  This package is the thin Python binding."""
from .binding import (  # noqa: F401
    BF16, F32, TAGS_FRAME, TAGS_PATH, Function, Graph, RdfError, ack_program, fact_program, fib_program, lib, primes_program, tak_program,
    tree_fold_program, tree_net_program, unpack_path_tag, sum_loop_program, pairs_loop_program, primes_loop_program,
    tri_program, topdown_program, find_program,
)
