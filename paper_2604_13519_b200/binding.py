"""Thin ctypes binding over the C ABI in include/toolspec.h.

Argument marshalling only: every step of the verify path runs in the library's CUDA kernels and
host C++.  PyTorch is used to allocate the caller-owned device / pinned buffers and to own the
stream.  There is no fallback: if the shared library is missing the import of `lib()` raises.
"""
import ctypes as C
import os
from typing import List, Optional, Sequence

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libtoolspec.so")
DEBUG_LIB_PATH = os.path.join(_HERE, "libtoolspec_dbg.so")   # built with every device-side index check compiled in

TS_K_MAX = 64
TS_PAGE_SIZE = 16
TS_FLAG_SKIP_LM_HEAD = 1
TS_FLAG_WANT_TOPK = 2
TS_TOPK = 8

STATUS = {0: "TS_OK", -1: "TS_ERR_ARG", -2: "TS_ERR_STATE", -3: "TS_ERR_OOM_PAGES",
          -4: "TS_ERR_K_TOO_LARGE", -5: "TS_ERR_TOKEN_RANGE", -6: "TS_ERR_DEVICE_TIMEOUT",
          -7: "TS_ERR_CUDA", -8: "TS_ERR_UNIMPLEMENTED", -9: "TS_ERR_DEVICE_BOUNDS"}

(TS_W_EMBED, TS_W_LM_HEAD, TS_W_FINAL_GAIN, TS_W_Q, TS_W_K, TS_W_V, TS_W_O, TS_W_GATE, TS_W_UP,
 TS_W_DOWN, TS_W_GAIN1, TS_W_GAIN2) = range(12)


class TsError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__(f"{STATUS.get(code, code)}: {msg}")
        self.code = code


class ts_model_config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "d_model", "n_q_heads", "n_kv_heads", "head_dim",
                                         "d_ffn", "vocab")] + \
               [("rope_theta", C.c_float), ("rms_eps", C.c_float)] + \
               [(n, C.c_int32) for n in ("max_pages", "max_batch", "k_max", "max_rows", "max_ctx",
                                         "act_split", "path")]


class ts_buffer_sizes(C.Structure):
    _fields_ = [(n, C.c_uint64) for n in ("weights_bytes", "kv_pool_bytes", "workspace_bytes",
                                          "host_io_bytes")]


class ts_buffers(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("weights", "kv_pool", "workspace", "host_io")]


class ts_vocab_layout(C.Structure):
    _fields_ = [("vocab", C.c_int32), ("eos", C.c_int32), ("tool_call", C.c_int32)] + \
               [(n, C.c_int32 * 8) for n in ("pfx", "mid", "kvsep", "nxt", "end")] + \
               [(n, C.c_int32) for n in ("pfx_len", "mid_len", "kvsep_len", "nxt_len", "end_len")]


class ts_draft_config(C.Structure):
    _fields_ = [("n_cap", C.c_int32), ("max_new_tokens", C.c_int32)]


class ts_verify_result(C.Structure):
    _fields_ = [("k", C.c_int32), ("accept_len", C.c_int32), ("n_emitted", C.c_int32),
                ("emitted", C.c_int32 * TS_K_MAX), ("argmax", C.c_int32 * TS_K_MAX),
                ("first_row", C.c_int32)]


class ts_session_info(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("cache_len", "pending", "n_output", "finished", "fsm_kind",
                                         "fsm_tool", "fsm_key", "n_pages")]


_P = C.c_void_p
_I32P = C.POINTER(C.c_int32)


class ts_attention_args(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_q_heads", "n_kv_heads", "head_dim", "batch", "pages_per_seq",
                                         "out_rows", "planes")] + \
               [("cu_rows_host", _I32P), ("seq_len_host", _I32P)] + \
               [(n, _P) for n in ("cu_rows", "seq_len", "block_table", "q", "k_pages", "v_pages", "out")]


_SIGNATURES = {
    "ts_query_buffer_sizes": [C.POINTER(ts_model_config), C.POINTER(ts_buffer_sizes)],
    "ts_init_model": [C.POINTER(ts_model_config), C.POINTER(ts_buffers), _P, C.POINTER(_P)],
    "ts_load_tensor": [_P, C.c_int32, C.c_int32, _P, C.c_int64, C.c_int64],
    "ts_model_destroy": [_P],
    "ts_schema_create": [C.POINTER(ts_vocab_layout), C.POINTER(_P)],
    "ts_schema_add_tool": [_P, _I32P, C.c_int32, _I32P, _I32P, C.c_int32],
    "ts_schema_destroy": [_P],
    "ts_datastore_create": [C.c_int32, C.POINTER(_P)],
    "ts_datastore_add": [_P, _I32P, C.c_int32, C.c_int32],
    "ts_datastore_attach_hidden": [_P, _P, C.c_int32, C.c_int32],
    "ts_datastore_add_hidden": [_P, _P, C.c_int32, _I32P, C.c_int32, C.c_int32],
    "ts_session_retrieve": [_P, _P, C.c_int32, C.c_int32, _P, _I32P, C.POINTER(C.c_float), _I32P],
    "ts_datastore_destroy": [_P],
    "ts_session_create": [_P, _P, _P, C.POINTER(ts_draft_config), C.POINTER(_P)],
    "ts_session_set_ranks": [_P, _I32P, C.c_int32],
    "ts_session_destroy": [_P],
    "ts_prefill": [_P, _P, _I32P, C.c_int32],
    "ts_draft": [_P, C.c_int32, _I32P, _I32P, _I32P],
    "ts_draft_tree": [_P, C.c_int32, _I32P, _I32P, _I32P, _I32P],
    "ts_verify": [_P, C.POINTER(_P), C.c_int32, _I32P, _I32P, C.c_uint32, C.POINTER(ts_verify_result)],
    "ts_verify_tree": [_P, C.POINTER(_P), C.c_int32, _I32P, _I32P, _I32P, C.c_uint32, C.POINTER(ts_verify_result),
                       _I32P],
    "ts_verify_sampled": [_P, C.POINTER(_P), C.c_int32, _I32P, _I32P, C.c_float, C.POINTER(C.c_float), C.c_uint32,
                          C.POINTER(ts_verify_result)],
    "ts_topk_cosine": [_P, _P, C.c_int32, _P, C.c_int32, C.c_int32, _P, _I32P, C.POINTER(C.c_float)],
    "ts_last_hidden": [_P, C.c_int32, C.POINTER(C.c_float)],
    "ts_session_enable_general_sd": [_P, C.c_int32],
    "ts_session_set_successors": [_P, C.c_int32, _I32P],
    "ts_session_successors": [_P, C.c_int32, _I32P, _I32P],
    "ts_last_topk": [_P, C.c_int32, _I32P, C.POINTER(C.c_float)],
    "ts_debug_restart": [_P, C.c_int32, C.c_int32],
    "ts_verify_tree_sampled": [_P, C.POINTER(_P), C.c_int32, _I32P, _I32P, _I32P, C.c_float, C.POINTER(C.c_float),
                               C.c_uint32, C.POINTER(ts_verify_result), _I32P],
    "ts_verify_replay": [_P],
    "ts_profile_step": [_P, C.POINTER(C.c_float), _I32P, C.c_int32],
    "ts_commit": [_P, C.POINTER(ts_verify_result)],
    "ts_commit_forced": [_P, _I32P, C.c_int32],
    "ts_session_state": [_P, C.POINTER(ts_session_info)],
    "ts_session_output": [_P, _I32P, C.c_int32, _I32P],
    "ts_debug_import_kv": [_P, _P, C.c_int32, _P, _P, C.c_int32],
    "ts_debug_export_kv": [_P, _P, C.c_int32, _P, _P, C.c_int32],
    "ts_debug_set_cache": [_P, C.c_int32, C.c_int32],
    "ts_read_logits": [_P, C.c_int32, C.c_int32, C.POINTER(C.c_float)],
    "ts_debug_read_buffer": [_P, C.c_int32, _P, C.c_uint64],
    "ts_debug_inject_device_error": [_P, C.c_int32],
    "ts_debug_timeline": [_P, C.POINTER(C.c_uint64), _I32P, C.c_int32, _I32P],
    "ts_model_counters": [_P, C.POINTER(C.c_int64), C.POINTER(C.c_int64), C.POINTER(C.c_int64)],
    "ts_attention_static": [C.POINTER(ts_attention_args), _P],
    "ts_debug_phase_clocks": [_P, C.POINTER(C.c_uint64), C.c_int32, _I32P],
    "ts_debug_schedule": [C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int32, _I32P, _I32P],
}
EXPORTED = sorted(list(_SIGNATURES) + ["ts_last_error"])

_lib = None


def use_debug_library():
    """Load the library's debug build (`python -m paper_2604_13519_b200.build --debug-bounds`) instead of the release
    one: the same code with every index a kernel takes from the step's inputs checked on the device; a failed check
    makes the step return TS_ERR_DEVICE_BOUNDS.  Has to be called before the library is first used in the process."""
    global LIB_PATH
    if _lib is not None:
        raise RuntimeError("the library is already loaded")
    LIB_PATH = DEBUG_LIB_PATH


def lib():
    """The loaded shared library.  Raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with "
                               f"`python -m paper_2604_13519_b200.build` (needs nvcc)")
        L = C.CDLL(LIB_PATH)
        for name, args in _SIGNATURES.items():
            fn = getattr(L, name)
            fn.argtypes = args
            fn.restype = C.c_int32
        L.ts_last_error.restype = C.c_char_p
        L.ts_last_error.argtypes = []
        _lib = L
    return _lib


def _check(code):
    if code != 0:
        raise TsError(code, lib().ts_last_error().decode())


def _i32(seq: Sequence[int]):
    arr = (C.c_int32 * max(1, len(seq)))(*seq)
    return arr


# ---- the same names as the C ABI, with Python-friendly arguments ----------------------------------
class Schema:
    def __init__(self, vocab_layout, tools):
        """vocab_layout: object with size, eos, tool_call, pfx, mid, kvsep, nxt, end;
        tools: iterable of objects with .name (ids) and .keys (list of id lists)."""
        v = ts_vocab_layout()
        v.vocab, v.eos, v.tool_call = vocab_layout.size, vocab_layout.eos, vocab_layout.tool_call
        for f in ("pfx", "mid", "kvsep", "nxt", "end"):
            ids = list(getattr(vocab_layout, f))
            setattr(v, f + "_len", len(ids))
            arr = getattr(v, f)
            for i, t in enumerate(ids):
                arr[i] = t
        self.h = _P()
        _check(lib().ts_schema_create(C.byref(v), C.byref(self.h)))
        self.n_tools = 0
        for t in tools:
            flat, offs = [], [0]
            for k in t.keys:
                flat += list(k)
                offs.append(len(flat))
            _check(lib().ts_schema_add_tool(self.h, _i32(t.name), len(t.name), _i32(flat), _i32(offs),
                                            len(t.keys)))
            self.n_tools += 1

    def __del__(self):
        if getattr(self, "h", None) and _lib is not None:
            _lib.ts_schema_destroy(self.h)
            self.h = None


class Datastore:
    def __init__(self, n_tools: int):
        self.h = _P()
        _check(lib().ts_datastore_create(n_tools, C.byref(self.h)))
        self.n = 0

    def add(self, tokens: Sequence[int], tool_id: int):
        _check(lib().ts_datastore_add(self.h, _i32(tokens), len(tokens), tool_id))
        self.n += 1

    def attach_hidden(self, hidden):
        """hidden: CUDA bf16 tensor [capacity][d_model], owned by the caller (kept referenced here)."""
        self.hidden = hidden
        if hidden is None:
            _check(lib().ts_datastore_attach_hidden(self.h, None, 0, 0))
        else:
            assert hidden.is_cuda and hidden.is_contiguous() and hidden.element_size() == 2
            _check(lib().ts_datastore_attach_hidden(self.h, _P(hidden.data_ptr()), hidden.shape[0], hidden.shape[1]))

    def add_hidden(self, model, row: int, tokens: Sequence[int], tool_id: int):
        """Append (h_j, y_j): h_j = final-norm hidden state of `row` of the model's last step."""
        _check(lib().ts_datastore_add_hidden(self.h, model.h, row, _i32(tokens), len(tokens), tool_id))
        self.n += 1

    def __del__(self):
        if getattr(self, "h", None) and _lib is not None:
            _lib.ts_datastore_destroy(self.h)
            self.h = None


class Model:
    """ts_init_model + ts_load_tensor over buffers allocated with torch."""

    def __init__(self, shape, max_pages: int, max_batch: int, k_max: int, max_rows: int, max_ctx: int,
                 act_split: bool = True, device="cuda:0", stream=None, path: int = 0):
        import torch
        self.torch = torch
        self.shape = shape
        c = ts_model_config()
        for n in ("n_layers", "d_model", "n_q_heads", "n_kv_heads", "head_dim", "d_ffn", "vocab",
                  "rope_theta", "rms_eps"):
            setattr(c, n, getattr(shape, n))
        c.max_pages, c.max_batch, c.k_max, c.max_rows, c.max_ctx = max_pages, max_batch, k_max, max_rows, max_ctx
        c.act_split = 1 if act_split else 0
        c.path = path
        self.cfg = c
        sizes = ts_buffer_sizes()
        _check(lib().ts_query_buffer_sizes(C.byref(c), C.byref(sizes)))
        self.sizes = sizes
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        mk = lambda n: torch.empty(int(n) + 1024, dtype=torch.uint8, device=self.device)
        self._raw = [mk(sizes.weights_bytes), mk(sizes.kv_pool_bytes), mk(sizes.workspace_bytes)]
        self._host = torch.empty(int(sizes.host_io_bytes), dtype=torch.uint8).pin_memory()
        al = lambda t: (t.data_ptr() + 1023) // 1024 * 1024
        self.kv_pool_ptr = al(self._raw[1])
        b = ts_buffers(al(self._raw[0]), self.kv_pool_ptr, al(self._raw[2]), self._host.data_ptr())
        self.stream = stream
        sp = stream.cuda_stream if stream is not None else torch.cuda.current_stream().cuda_stream
        self.stream_ptr = sp
        self.h = _P()
        _check(lib().ts_init_model(C.byref(c), C.byref(b), _P(sp), C.byref(self.h)))

    def kv_pool_tensor(self):
        """The caller-owned KV pool viewed as an fp16 tensor (e.g. to fill it with synthetic data)."""
        torch = self.torch
        off = self.kv_pool_ptr - self._raw[1].data_ptr()
        n = int(self.sizes.kv_pool_bytes)
        return self._raw[1][off:off + n].view(torch.float16)

    def load_tensor(self, kind: int, layer: int, t):
        t = t.contiguous()
        rows, cols = (t.shape if t.dim() == 2 else (1, t.shape[0]))
        _check(lib().ts_load_tensor(self.h, kind, layer, _P(t.data_ptr()), rows, cols))

    def load_weights(self, w: dict):
        """w: name -> CPU tensor, names as produced by the synthetic generator."""
        self.load_tensor(TS_W_EMBED, 0, w["embed"])
        self.load_tensor(TS_W_LM_HEAD, 0, w["lm_head"])
        self.load_tensor(TS_W_FINAL_GAIN, 0, w["gf"].float())
        kinds = dict(wq=TS_W_Q, wk=TS_W_K, wv=TS_W_V, wo=TS_W_O, wg=TS_W_GATE, wu=TS_W_UP, wd=TS_W_DOWN,
                     g1=TS_W_GAIN1, g2=TS_W_GAIN2)
        for l in range(self.shape.n_layers):
            for n, kind in kinds.items():
                t = w[f"l{l}.{n}"]
                self.load_tensor(kind, l, t.float() if n[0] == "g" else t)

    def read_logits(self, row0: int, n_rows: int):
        import numpy as np
        out = np.empty((n_rows, self.cfg.vocab), dtype=np.float32)
        _check(lib().ts_read_logits(self.h, row0, n_rows, out.ctypes.data_as(C.POINTER(C.c_float))))
        return out

    def read_buffer(self, which: int):
        """Internal activation buffer `which` of the last step as a CPU tensor (test support)."""
        torch = self.torch
        s, R = self.shape, (self.cfg.max_rows + 127) // 128 * 128
        P = 1 + self.cfg.act_split
        Nq = s.n_q_heads * s.head_dim
        shape, dt = {0: ((R, s.d_model), torch.float32), 1: ((P, R, s.d_model), torch.bfloat16),
                     2: ((R, Nq), torch.float16), 3: ((P, R, Nq), torch.bfloat16),
                     4: ((P, R, s.d_ffn), torch.bfloat16)}[which]
        out = torch.empty(shape, dtype=dt)
        _check(lib().ts_debug_read_buffer(self.h, which, _P(out.data_ptr()), out.numel() * out.element_size()))
        return out

    def phase_clocks(self):
        """[3][n_phases] device clocks (ns) left by the last ts_profile_step of the persistent kernel."""
        import numpy as np
        n = C.c_int32()
        buf = (C.c_uint64 * 4096)()
        _check(lib().ts_debug_phase_clocks(self.h, buf, 4096, C.byref(n)))
        return np.array(buf[:3 * n.value], dtype=np.uint64).reshape(3, n.value)

    def timeline(self):
        """[(class name, start, first wait return, last wait return, end)] per launch of the last step re-run under
        its normal launch configuration; times in microseconds from the first kernel's start."""
        cap = 9 * self.shape.n_layers + 16
        st = (C.c_uint64 * (4 * cap))()
        cls = (C.c_int32 * cap)()
        n = C.c_int32(0)
        _check(lib().ts_debug_timeline(self.h, st, cls, cap, C.byref(n)))
        rows, t0 = [], None
        for i in range(min(n.value, cap)):
            v = [st[4 * i + j] for j in range(4)]
            if v[3] == 0:
                continue
            t0 = v[0] if t0 is None else t0
            rows.append((KERNEL_CLASSES[cls[i]],) + tuple((x - t0) / 1e3 for x in v))
        return rows

    def inject_device_error(self, code: int):
        """Test support: the next step reports `code` in its device status word (see toolspec.h)."""
        _check(lib().ts_debug_inject_device_error(self.h, code))

    def counters(self):
        a, b, c = C.c_int64(), C.c_int64(), C.c_int64()
        _check(lib().ts_model_counters(self.h, C.byref(a), C.byref(b), C.byref(c)))
        return a.value, b.value, c.value

    def close(self):
        if getattr(self, "h", None):
            lib().ts_model_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class Session:
    def __init__(self, model: Optional[Model], schema: Optional[Schema], store: Optional[Datastore],
                 n_cap: int = 32, max_new_tokens: int = 1 << 30):
        self.model, self.schema, self.store = model, schema, store      # keep handles alive
        cfg = ts_draft_config(n_cap, max_new_tokens)
        self.h = _P()
        _check(lib().ts_session_create(model.h if model else None, schema.h if schema else None,
                                       store.h if store else None, C.byref(cfg), C.byref(self.h)))

    def enable_general_sd(self, on: bool = True):
        _check(lib().ts_session_enable_general_sd(self.h, 1 if on else 0))

    def set_successors(self, token: int, ids: Sequence[int]):
        assert len(ids) == TS_TOPK
        _check(lib().ts_session_set_successors(self.h, token, _i32(ids)))

    def successors(self, token: int):
        ids = (C.c_int32 * TS_TOPK)()
        found = C.c_int32(0)
        _check(lib().ts_session_successors(self.h, token, ids, C.byref(found)))
        return list(ids) if found.value else None

    def set_ranks(self, ranks: Sequence[int]):
        _check(lib().ts_session_set_ranks(self.h, _i32(ranks), len(ranks)))

    def state(self) -> ts_session_info:
        info = ts_session_info()
        _check(lib().ts_session_state(self.h, C.byref(info)))
        return info

    def output(self) -> List[int]:
        n = C.c_int32()
        _check(lib().ts_session_output(self.h, None, 0, C.byref(n)))
        buf = (C.c_int32 * max(1, n.value))()
        _check(lib().ts_session_output(self.h, buf, n.value, C.byref(n)))
        return list(buf[:n.value])

    def set_cache(self, cache_len: int, pending: int):
        _check(lib().ts_debug_set_cache(self.h, cache_len, pending))

    def restart(self, cache_len: int, pending: int):
        _check(lib().ts_debug_restart(self.h, cache_len, pending))

    def import_kv(self, layer: int, k, v):
        """k, v: CPU tensors [n_tokens][n_kv_heads][head_dim] (any float dtype; sent as float32)."""
        k, v = k.float().contiguous(), v.float().contiguous()
        _check(lib().ts_debug_import_kv(self.model.h, self.h, layer, _P(k.data_ptr()), _P(v.data_ptr()),
                                        k.shape[0]))

    def export_kv(self, layer: int, n_tokens: int):
        torch = self.model.torch
        s = self.model.shape
        k = torch.empty(n_tokens, s.n_kv_heads, s.head_dim, dtype=torch.float32)
        v = torch.empty_like(k)
        _check(lib().ts_debug_export_kv(self.model.h, self.h, layer, _P(k.data_ptr()), _P(v.data_ptr()),
                                        n_tokens))
        return k, v

    def close(self):
        if getattr(self, "h", None):
            lib().ts_session_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def ts_prefill(model: Optional[Model], session: Session, tokens: Sequence[int]):
    _check(lib().ts_prefill(model.h if model else None, session.h, _i32(tokens), len(tokens)))


def ts_draft(session: Session, max_draft: int):
    """Returns (draft ids, source) with source 0 none, 1 schema FSM, 2 retrieval."""
    buf = (C.c_int32 * max(1, max_draft))()
    n, src = C.c_int32(), C.c_int32()
    _check(lib().ts_draft(session.h, max_draft, buf, C.byref(n), C.byref(src)))
    return list(buf[:n.value]), src.value


def ts_verify(model: Model, sessions: Sequence[Session], drafts: Sequence[Sequence[int]], flags: int = 0):
    """Returns a list of ts_verify_result, one per session."""
    B = len(sessions)
    hs = (_P * B)(*[s.h for s in sessions])
    flat, offs = [], [0]
    for d in drafts:
        flat += list(d)
        offs.append(len(flat))
    out = (ts_verify_result * B)()
    _check(lib().ts_verify(model.h, hs, B, _i32(flat), _i32(offs), flags, out))
    return list(out)


def ts_draft_tree(session: Session, max_nodes: int):
    """(tokens of nodes 1.., parent node of each of them, source)."""
    toks = (C.c_int32 * TS_K_MAX)()
    par = (C.c_int32 * TS_K_MAX)()
    n, src = C.c_int32(0), C.c_int32(0)
    _check(lib().ts_draft_tree(session.h, max_nodes, toks, par, C.byref(n), C.byref(src)))
    return list(toks[:n.value]), list(par[:n.value]), src.value


def ts_verify_tree(model: Model, sessions: Sequence[Session], drafts: Sequence[Sequence[int]],
                   parents: Sequence[Sequence[int]], flags: int = 0):
    """Draft trees: drafts[i][j] is node j+1 of sequence i, parents[i][j] its parent node (0 = the pending
    token).  Returns (list of ts_verify_result, list of accepted paths as node indices, root first)."""
    B = len(sessions)
    hs = (_P * B)(*[s.h for s in sessions])
    flat, par, offs = [], [], [0]
    for d, p in zip(drafts, parents):
        assert len(d) == len(p)
        flat += list(d)
        par += list(p)
        offs.append(len(flat))
    out = (ts_verify_result * B)()
    path = (C.c_int32 * (B * TS_K_MAX))()
    _check(lib().ts_verify_tree(model.h, hs, B, _i32(flat), _i32(par), _i32(offs), flags, out, path))
    paths = [[path[i * TS_K_MAX + j] for j in range(out[i].accept_len + 1)] for i in range(B)]
    return list(out), paths


def ts_verify_sampled(model: Model, sessions: Sequence[Session], drafts: Sequence[Sequence[int]],
                      temperature: float, uniforms: Sequence[float], flags: int = 0):
    """Speculative-sampling acceptance; uniforms: one value in [0, 1) per chunk row, chunk after chunk."""
    B = len(sessions)
    hs = (_P * B)(*[s.h for s in sessions])
    flat, offs = [], [0]
    for d in drafts:
        flat += list(d)
        offs.append(len(flat))
    assert len(uniforms) == len(flat) + B
    u = (C.c_float * len(uniforms))(*uniforms)
    out = (ts_verify_result * B)()
    _check(lib().ts_verify_sampled(model.h, hs, B, _i32(flat), _i32(offs), temperature, u, flags, out))
    return list(out)


def ts_topk_cosine(model: Model, hidden, K: int, query=None, row: int = 0):
    """hidden: CUDA bf16 tensor [N][d]; query: CUDA float32 tensor [d] or None (hidden state of `row` of the last
    step).  Returns (indices, scores), best first."""
    torch = model.torch
    N = hidden.shape[0]
    assert hidden.is_cuda and hidden.dtype == torch.bfloat16 and hidden.is_contiguous()
    scratch = torch.empty(N + 2 * K + 1 + 2 * K * ((N + 4095) // 4096), dtype=torch.float32, device=hidden.device)
    idx = (C.c_int32 * K)()
    sc = (C.c_float * K)()
    q = _P(query.data_ptr()) if query is not None else None
    _check(lib().ts_topk_cosine(model.h, _P(hidden.data_ptr()), N, q, row, K, _P(scratch.data_ptr()), idx, sc))
    return list(idx), list(sc)


def ts_session_retrieve(model: Model, session: Session, K: int, row: int = 0):
    """Algorithm 1's once-per-query step: h_x (row of the last step) -> Top-K over the datastore's hidden states ->
    installed as the session's candidate order.  Returns (indices, scores), best first."""
    torch = model.torch
    N = session.store.n
    k = max(1, min(K, N, 64))
    scratch = torch.empty(N + 2 * k + 1 + 2 * k * ((N + 4095) // 4096), dtype=torch.float32, device=model.device)
    idx = (C.c_int32 * 64)()
    sc = (C.c_float * 64)()
    nk = C.c_int32(0)
    _check(lib().ts_session_retrieve(model.h, session.h, row, K, _P(scratch.data_ptr()), idx, sc, C.byref(nk)))
    return list(idx[:nk.value]), list(sc[:nk.value])


def ts_last_hidden(model: Model, row: int):
    import numpy as np
    out = np.empty(model.cfg.d_model, dtype=np.float32)
    _check(lib().ts_last_hidden(model.h, row, out.ctypes.data_as(C.POINTER(C.c_float))))
    return out


def ts_last_topk(model: Model, row: int):
    ids = (C.c_int32 * TS_TOPK)()
    vals = (C.c_float * TS_TOPK)()
    _check(lib().ts_last_topk(model.h, row, ids, vals))
    return list(ids), list(vals)


def ts_verify_tree_sampled(model: Model, sessions: Sequence[Session], drafts: Sequence[Sequence[int]],
                           parents: Sequence[Sequence[int]], temperature: float, uniforms: Sequence[float],
                           flags: int = 0):
    """Draft trees accepted by speculative sampling; uniforms: one value per chunk node (value 0 of a chunk draws
    the sample).  Returns (results, accepted paths)."""
    B = len(sessions)
    hs = (_P * B)(*[s.h for s in sessions])
    flat, par, offs = [], [], [0]
    for d, p in zip(drafts, parents):
        flat += list(d)
        par += list(p)
        offs.append(len(flat))
    assert len(uniforms) == len(flat) + B
    u = (C.c_float * len(uniforms))(*uniforms)
    out = (ts_verify_result * B)()
    path = (C.c_int32 * (B * TS_K_MAX))()
    _check(lib().ts_verify_tree_sampled(model.h, hs, B, _i32(flat), _i32(par), _i32(offs), temperature, u, flags, out,
                                        path))
    return list(out), [[path[i * TS_K_MAX + j] for j in range(out[i].accept_len + 1)] for i in range(B)]


def ts_verify_replay(model: Model):
    _check(lib().ts_verify_replay(model.h))


KERNEL_CLASSES = ("gemm", "attention", "attention_merge", "norm", "rope_kv", "accept", "fused_kernel")


def ts_profile_step(model: Model):
    """dict class -> (total ms, launches) for one replay of the last step, kernels serialised."""
    ms = (C.c_float * 8)()
    n = (C.c_int32 * 8)()
    _check(lib().ts_profile_step(model.h, ms, n, 8))
    return {k: (ms[i], n[i]) for i, k in enumerate(KERNEL_CLASSES)}


def ts_commit(session: Session, result: ts_verify_result):
    _check(lib().ts_commit(session.h, C.byref(result)))


def ts_commit_forced(session: Session, emitted: Sequence[int]):
    _check(lib().ts_commit_forced(session.h, _i32(emitted), len(emitted)))


def ts_attention_static(q, k_pages, v_pages, block_table, cu_rows: Sequence[int], seq_len: Sequence[int],
                        n_q_heads: int, n_kv_heads: int, head_dim: int, out, stream=None, cu_rows_dev=None,
                        seq_len_dev=None):
    """Attention stage of the verify step with library-resident scratch (no device allocation in the
    call).  q, k_pages, v_pages: CUDA fp16 tensors; block_table: CUDA int32 [batch][pages_per_seq];
    cu_rows / seq_len: Python ints; their device copies (int32 CUDA tensors) are taken from cu_rows_dev /
    seq_len_dev, or made here (an allocation by this wrapper, not by the library call) when those are None;
    out: CUDA bf16 tensor [planes][out_rows][n_q_heads*head_dim], written in place."""
    import torch
    B = len(seq_len)
    a = ts_attention_args()
    a.n_q_heads, a.n_kv_heads, a.head_dim = n_q_heads, n_kv_heads, head_dim
    a.batch, a.pages_per_seq = B, block_table.shape[1]
    a.planes, a.out_rows = out.shape[0], out.shape[1]
    h_cu, h_len = _i32(cu_rows), _i32(seq_len)
    d_cu = cu_rows_dev if cu_rows_dev is not None else torch.tensor(list(cu_rows), dtype=torch.int32, device=q.device)
    d_len = seq_len_dev if seq_len_dev is not None else torch.tensor(list(seq_len), dtype=torch.int32, device=q.device)
    a.cu_rows_host, a.seq_len_host = h_cu, h_len
    a.cu_rows, a.seq_len, a.block_table = d_cu.data_ptr(), d_len.data_ptr(), block_table.data_ptr()
    a.q, a.k_pages, a.v_pages, a.out = q.data_ptr(), k_pages.data_ptr(), v_pages.data_ptr(), out.data_ptr()
    sp = stream.cuda_stream if stream is not None else torch.cuda.current_stream().cuda_stream
    _check(lib().ts_attention_static(C.byref(a), _P(sp)))
    return d_cu, d_len      # keep the device copies alive until the caller has synchronised
