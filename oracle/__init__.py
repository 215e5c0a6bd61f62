"""CPU oracle for the KVCompose compression pass -- test infrastructure only.

Nothing in the product package imports this.  See ``kvc_oracle.c`` for the
arithmetic and ``api.py`` for the numpy-facing wrappers.
"""
from .api import (  # noqa: F401
    AGG_MAX,
    AGG_MEAN,
    allocate,
    allocate_floor,
    attention_rows,
    budget_from_ratio,
    build,
    compose,
    compose_f32,
    compress,
    gather_layer,
    get_threads,
    has_openmp,
    rank,
    score_layer,
    score_layer_vnorm,
    select_unstructured,
    set_threads,
    sort_kept,
)
