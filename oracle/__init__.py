"""Independent CPU oracle (float64) for the ToolSpec verify path and its drafters.

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the benchmark's CPU-baseline
leg.  The product package never imports it and shares no code with it.
"""
from .transformer import (OracleModel, KVCache, rmsnorm, rope, attention, swiglu,   # noqa: F401
                          argmax_lowest, top2_gap, topk_lowest)
from .drafter import (SchemaFsm, Datastore, Drafter, suffix_match, suffix_matches, validate_prefix,   # noqa: F401
                      context_match, recycled_tree, RECYCLE_TREE, TOPK,
                      Q_O, Q_T, Q_P, Q_V, Q_DONE, SUFFIX_LENGTHS, DEFAULT_N_CAP)
from .loop import prefill, vanilla_greedy, speculative_decode, speculative_decode_tree  # noqa: F401
from .tree import (verify_tree, forward_tree, accepted_path, ancestor_mask, node_depths,  # noqa: F401
                   pack_candidates)
from .sampling import (target_probs, sample_inverse_cdf, accept_sampled, verify_sampled,   # noqa: F401
                       accept_sampled_tree)
from .retrieval import cosine_scores, topk_cosine, HiddenStore   # noqa: F401
