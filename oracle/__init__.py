"""CPU oracle for the PRISM hot path.  TEST INFRASTRUCTURE ONLY.

A plain, slow, fp64 numpy restatement of what the hot path computes: the per-candidate
cross-encoder forward (decoder stack in reranker.py, encoder stack in encoder.py) with
intermediate score probes (Sec. 3.1, 4.1 of the paper) and the
progressive cluster-pruning rule replayed over those scores (Sec. 4.1, 4.5).  It shares no
code with the CUDA path and must never be imported by it: only tests/, the smoke check and
the bench's cpu_baseline leg may import this package.
"""
from .reranker import (rmsnorm, rope_rotate, attention, layer_forward,  # noqa: F401
                       candidate_scores, score_matrix)
from .encoder import (layernorm, gelu, embed_tokens, encoder_layer_forward, head_score,  # noqa: F401
                      encoder_candidate_scores, encoder_score_matrix)
from .quant import unpack_w4, dequantize_w4, dequantize_weights  # noqa: F401
from .prune_rule import (coefficient_of_variation, rank_order, optimal_partition,  # noqa: F401
                         route_clusters, replay_select, MODE_NONE, MODE_FIXED_KEEP, MODE_CLUSTER)
from .select import oracle_select  # noqa: F401
from .calibrate import Calibrator, calibrated_step, precision_at_k  # noqa: F401
