"""CPU oracle for the link-prediction training step -- TEST INFRASTRUCTURE ONLY.

A plain FP64 restatement of what the step computes (encoder of Eq. 1, edge predictor of
Eq. 2, the mean binary cross-entropy of Algorithm 1, its analytic gradient, gradient
averaging and the Adam update), plus integer-exact samplers.  It shares no code with the
CUDA library and must never be imported by it: only tests, the smoke check and the CPU
baseline leg of the benchmark use it.

Pin status (tests/test_oracle_*.py): every function below is pinned by closed forms,
dense brute force, finite differences or published known-answer vectors, except
  * accuracy (Hits@K) against the paper's tables -- parity unpinned (needs the public
    datasets, which are not available).
"""
from .build import lib, build_oracle  # noqa: F401
from .sparse import (  # noqa: F401
    philox4x32_10,
    csc_transpose,
    gcn_degree,
    aggregate,
    aggregate_backward,
    sample_negatives,
    sample_neighbors,
    build_blocks,
    sparsify,
    sparsified_graph,
    worker_view,
)
from .model import (  # noqa: F401
    split_params,
    forward,
    bce_with_logits,
    train_step,
    score,
    adam_step,
    average_gradients,
    hits_at_k,
    encoder_param_count,
    split_predictor,
)
