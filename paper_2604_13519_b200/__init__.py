"""B200-native verify path of ToolSpec (schema-aware, retrieval-augmented speculative decoding).

The product is the C-ABI shared library built from csrc/ (see include/toolspec.h); this package holds
its ctypes binding and the in-tree build step.  Importing the package does not load the library;
`binding.lib()` does, and raises if it has not been built.
"""
from . import binding                     # noqa: F401
from .binding import (Model, Schema, Datastore, Session, TsError, ts_prefill, ts_draft, ts_verify,   # noqa: F401
                      ts_verify_tree, ts_draft_tree, ts_verify_sampled, ts_verify_tree_sampled, ts_topk_cosine, ts_session_retrieve, ts_last_hidden, ts_last_topk, TS_FLAG_WANT_TOPK, TS_TOPK,
                      ts_verify_replay, ts_profile_step, ts_commit, ts_commit_forced, ts_attention_static, TS_FLAG_SKIP_LM_HEAD, TS_K_MAX)
