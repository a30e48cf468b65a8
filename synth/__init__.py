"""Seeded synthetic inputs shared by the CPU oracle's tests and the CUDA path's tests.

This package only *produces data* (model shapes, weight blobs, schemas, historical
invocations, contexts, synthetic KV, corrupted drafts).  It contains none of the method's
arithmetic: no forward pass, no finite-state machine, no suffix matching, no acceptance rule.
"""
from .shapes import ModelShape, SHAPES, MASTER_SEED          # noqa: F401
from .weights import make_weights, tensor_names              # noqa: F401
from .toolcalls import (Vocab, Schema, Tool, make_schema, make_datastore,   # noqa: F401
                        make_context, render_invocation, zipf_tool_ids)
from .kv import make_synthetic_kv                            # noqa: F401
