"""ctypes binding of libtasc.so: argument marshalling only.

Every function mirrors the C entry point of the same name in ``include/tasc.h``; tensors are
torch CUDA tensors used as device buffers, and every step of the path runs inside the library's
kernels.  Importing this module fails loudly if the library has not been built.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
from . import LIBRARY_FILE            # "libtasc.so"; timeline.py switches to the instrumented build of the same sources
LIB_PATH = os.path.join(_HERE, LIBRARY_FILE)

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2602_24174_b200.build` "
        "(there is no CPU or PyTorch fallback for this path)")

lib = C.CDLL(LIB_PATH)

OK, EINVAL, ENOMEM, ECUDA, ECAPACITY, ENOKV, ETIMEOUT = 0, -1, -2, -3, -4, -5, -6
MAX_ORDER, MAX_ROWS, VOCAB_BITS, TOK_MAX_N = 5, 16, 20, 6
F32, BF16 = 0, 1
MODE_GREEDY, MODE_CONTINUATION, MODE_FORCED_ACCEPT = 0, 1, 2


class TascError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        detail = lib.tasc_last_error().decode() if code == ECUDA else ""
        super().__init__(f"{where}: {lib.tasc_status_string(code).decode()} ({code})" + (f": {detail}" if detail else ""))


class NgramEntry(C.Structure):
    _fields_ = [("n", C.c_int32), ("ctx", C.c_int32 * MAX_ORDER), ("next", C.c_int32), ("count", C.c_uint32)]


class ModelDesc(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("d_model", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("d_ff", C.c_int32), ("vocab", C.c_int32), ("dtype", C.c_int32),
                ("rope_base", C.c_float), ("rms_eps", C.c_float), ("max_positions", C.c_int32), ("page_size", C.c_int32)]


class Weights(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("lm_head", C.c_void_p), ("final_norm", C.c_void_p),
                ("attn_norm", C.POINTER(C.c_void_p)), ("wqkv", C.POINTER(C.c_void_p)), ("wo", C.POINTER(C.c_void_p)),
                ("mlp_norm", C.POINTER(C.c_void_p)), ("w_gate_up", C.POINTER(C.c_void_p)), ("w_down", C.POINTER(C.c_void_p))]


class Kv(C.Structure):
    _fields_ = [("pool", C.c_void_p), ("n_pages", C.c_int64), ("block_table", C.c_void_p), ("max_pages_per_seq", C.c_int32)]


class Seqs(C.Structure):
    _fields_ = [("tokens", C.c_void_p), ("stride", C.c_int64), ("len", C.c_void_p), ("stop_len", C.c_void_p)]


class CorpusStatistics(C.Structure):
    _fields_ = [("n_tokens", C.c_int64), ("n_bigrams", C.c_int64), ("n_unique_tokens", C.c_int64), ("n_unique_bigrams", C.c_int64),
                ("bigrams_for_cdf", C.c_int64), ("bigram_entropy_bits", C.c_double), ("typical_set_size", C.c_double),
                ("token_entropy_bits", C.c_double), ("token_entropy_normalised", C.c_double), ("token_renyi2_bits", C.c_double)]


class DraftParams(C.Structure):
    _fields_ = [("k", C.c_int32), ("lambda_num", C.c_int32), ("lambda_den", C.c_int32), ("mode", C.c_int32),
                ("forced_accept", C.c_int32), ("continuation", C.c_void_p), ("continuation_stride", C.c_int64)]


class Stats(C.Structure):
    _fields_ = [("steps", C.c_int64), ("committed", C.c_int64), ("accepted_hist", C.c_int64 * MAX_ROWS),
                ("prefill_ms", C.c_float), ("decode_ms", C.c_float)]


_P = C.c_void_p
lib.tasc_status_string.restype = C.c_char_p
lib.tasc_status_string.argtypes = [C.c_int32]
lib.tasc_last_error.restype = C.c_char_p
lib.tasc_drafter_build.argtypes = [_P, _P, C.c_int64, C.c_int32, C.c_int32, C.c_int32, _P, C.POINTER(_P)]
lib.tasc_drafter_export.argtypes = [_P, C.POINTER(NgramEntry), C.c_int64, C.POINTER(C.c_int64), C.POINTER(C.c_int32)]
lib.tasc_drafter_destroy.argtypes = [_P]
lib.tasc_drafter_import.argtypes = [C.POINTER(NgramEntry), C.c_int64, C.c_int32, C.c_int32, C.c_int32, _P, C.POINTER(_P)]
lib.tasc_drafter_import.restype = C.c_int32
lib.tasc_drafter_from_bigram.argtypes = [_P, C.c_int32, _P, C.POINTER(_P)]
lib.tasc_drafter_from_bigram.restype = C.c_int32
lib.tasc_bigram_table.argtypes = [_P, C.POINTER(Kv), C.c_int32, _P, _P, C.c_size_t, _P]
lib.tasc_bigram_table.restype = C.c_int32
lib.tasc_tok_enrich.argtypes = [_P, _P, C.c_int64, C.c_int32, C.c_int32, C.c_int32, _P, C.POINTER(C.c_int32), _P, _P, _P]
lib.tasc_tok_enrich.restype = C.c_int32
lib.tasc_tok_init_rows.argtypes = [_P, C.c_int32, C.c_int32, C.c_int32, _P, C.c_int32, _P, _P, _P]
lib.tasc_tok_init_rows.restype = C.c_int32
lib.tasc_tok_encode.argtypes = [_P, _P, C.c_int64, C.c_int32, _P, C.c_int32, _P, _P, _P]
lib.tasc_tok_encode.restype = C.c_int32
lib.tasc_corpus_stats.argtypes = [_P, _P, C.c_int64, C.c_int32, C.c_int32, C.c_int32, _P, C.POINTER(CorpusStatistics)]
lib.tasc_corpus_stats.restype = C.c_int32
lib.tasc_draft.argtypes = [_P, _P, C.c_int64, _P, C.c_int32, C.c_int32, C.c_int32, C.c_int32, _P, _P]
lib.tasc_model_create.argtypes = [C.POINTER(ModelDesc), C.POINTER(Weights), C.POINTER(_P)]
lib.tasc_model_destroy.argtypes = [_P]
lib.tasc_workspace_bytes.restype = C.c_size_t
lib.tasc_workspace_bytes.argtypes = [_P, C.c_int32, C.c_int32]
lib.tasc_prefill.argtypes = [_P, C.POINTER(Kv), C.POINTER(Seqs), C.c_int32, C.c_int32, _P, C.c_size_t, _P]
lib.tasc_verify_step.argtypes = [_P, C.POINTER(Kv), C.POINTER(Seqs), _P, C.c_int32, C.c_int32, _P, _P, _P, _P, _P, _P,
                                 C.c_size_t, _P]
lib.tasc_generate.argtypes = [_P, _P, C.POINTER(Kv), C.POINTER(Seqs), C.c_int32, C.c_int32, C.POINTER(DraftParams), _P,
                              C.POINTER(Stats), _P, C.c_size_t, _P]
lib.tasc_poll_status.argtypes = [_P, _P]
lib.tasc_selftest_bounded_wait.argtypes = [_P, C.c_int64, _P]
lib.tasc_selftest_bounded_wait.restype = C.c_int32
lib.tasc_gemm_bf16.argtypes = [_P, _P, _P, C.c_int32, C.c_int32, C.c_int32, _P, C.c_size_t, _P]
lib.tasc_gemm_bf16x2.argtypes = [_P, _P, _P, C.c_int32, C.c_int32, C.c_int32, _P, C.c_size_t, _P]
lib.tasc_gemm_bf16x2.restype = C.c_int32
lib.tasc_gemm_bf16_static.argtypes = [_P, _P, _P, C.c_int32, C.c_int32, C.c_int32, _P, _P]
lib.tasc_gemm_bf16_static.restype = C.c_int32
lib.tasc_gemm_workspace_bytes.restype = C.c_size_t
lib.tasc_gemm_workspace_bytes.argtypes = [C.c_int32, C.c_int32, C.c_int32]
for _f in ("tasc_drafter_build", "tasc_drafter_export", "tasc_drafter_destroy", "tasc_draft", "tasc_model_create",
           "tasc_model_destroy", "tasc_prefill", "tasc_verify_step", "tasc_generate", "tasc_poll_status", "tasc_gemm_bf16"):
    getattr(lib, _f).restype = C.c_int32


lib.tasc_profile_kinds.restype = C.c_int32
lib.tasc_profile_kind_name.restype = C.c_char_p
lib.tasc_profile_kind_name.argtypes = [C.c_int32]
lib.tasc_profile_enable.argtypes = [C.c_int32]
lib.tasc_profile_enable.restype = C.c_int32
lib.tasc_profile_read.argtypes = [C.POINTER(C.c_double), C.POINTER(C.c_int64), C.c_int32]
lib.tasc_profile_read.restype = C.c_int32
lib.tasc_launch_counts.argtypes = [C.POINTER(C.c_int64), C.c_int32]
lib.tasc_launch_counts.restype = C.c_int32


def _check(code: int, where: str):
    if code != OK:
        raise TascError(code, where)


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _dev(t: torch.Tensor, dtype) -> torch.Tensor:
    assert t.is_cuda and t.dtype == dtype and t.is_contiguous(), (t.device, t.dtype, t.is_contiguous())
    return t


class Drafter:
    """tasc_drafter handle: corpus n-gram tables on the device."""

    def __init__(self, handle, n_max: int):
        self._h, self.n_max = handle, n_max

    def __del__(self):
        if getattr(self, "_h", None) and lib is not None:      # lib is None while the interpreter shuts down
            lib.tasc_drafter_destroy(self._h)
            self._h = None

    def export(self):
        """(entries as int64[E, MAX_ORDER + 3] rows (n, ctx padded with -1, next, count), fallback token)."""
        n = C.c_int64(0)
        fb = C.c_int32(0)
        _check(lib.tasc_drafter_export(self._h, None, 0, C.byref(n), C.byref(fb)), "tasc_drafter_export")
        buf = (NgramEntry * max(n.value, 1))()
        _check(lib.tasc_drafter_export(self._h, buf, n.value, C.byref(n), C.byref(fb)), "tasc_drafter_export")
        raw = np.frombuffer(buf, dtype=np.int32).reshape(-1, MAX_ORDER + 3)[:n.value]
        out = raw.astype(np.int64)
        out[:, MAX_ORDER + 2] = raw[:, MAX_ORDER + 2].view(np.uint32)
        return out, fb.value


def tasc_drafter_build(corpus_tokens: torch.Tensor, doc_offsets: torch.Tensor, n_max: int, p_min: int, vocab: int) -> Drafter:
    _dev(corpus_tokens, torch.int32)
    _dev(doc_offsets, torch.int64)
    h = _P()
    _check(lib.tasc_drafter_build(_ptr(corpus_tokens), _ptr(doc_offsets), doc_offsets.numel() - 1, n_max, p_min, vocab,
                                  _stream(), C.byref(h)), "tasc_drafter_build")
    return Drafter(h, n_max)


def tasc_drafter_import(entries: np.ndarray, fallback: int, n_max: int, vocab: int) -> Drafter:
    """Drafter handle from the array Drafter.export() returns (int64[E, MAX_ORDER + 3] rows n, ctx, next, count)."""
    entries = np.asarray(entries, dtype=np.int64).reshape(-1, MAX_ORDER + 3)
    buf = (NgramEntry * max(len(entries), 1))()
    raw = np.frombuffer(buf, dtype=np.int32).reshape(-1, MAX_ORDER + 3)
    raw[:len(entries), :MAX_ORDER + 2] = entries[:, :MAX_ORDER + 2]
    raw[:len(entries), MAX_ORDER + 2] = entries[:, MAX_ORDER + 2].astype(np.uint32).view(np.int32)
    h = _P()
    _check(lib.tasc_drafter_import(buf, len(entries), n_max, vocab, fallback, _stream(), C.byref(h)), "tasc_drafter_import")
    return Drafter(h, n_max)


def tasc_drafter_from_bigram(table: torch.Tensor, vocab: int) -> Drafter:
    """Drafter handle of the model-derived bigram (context token c -> table[c])."""
    _dev(table, torch.int32)
    assert table.numel() == vocab
    h = _P()
    _check(lib.tasc_drafter_from_bigram(_ptr(table), vocab, _stream(), C.byref(h)), "tasc_drafter_from_bigram")
    return Drafter(h, 1)


def tasc_bigram_table(model: "Model", kv: "Kv", B: int, workspace: torch.Tensor, out: torch.Tensor | None = None) -> torch.Tensor:
    """table[t] = the model's most probable next token after the single-token context t (int32[vocab] CUDA tensor)."""
    if out is None:
        out = torch.empty(model.shape.vocab, dtype=torch.int32, device=workspace.device)
    _dev(out, torch.int32)
    _check(lib.tasc_bigram_table(model._h, C.byref(kv), B, _ptr(out), _ptr(workspace), workspace.numel(), _stream()),
           "tasc_bigram_table")
    return out


def tasc_tok_enrich(corpus_tokens: torch.Tensor, doc_offsets: torch.Tensor, base_vocab: int, budget: int, n_max: int):
    """Algorithm 1.  Returns (merges int32[n_merges, TOK_MAX_N] padded with -1, tokens, offsets) as CUDA tensors."""
    _dev(corpus_tokens, torch.int32)
    _dev(doc_offsets, torch.int64)
    dev = doc_offsets.device
    merges = torch.empty((max(budget, 1), TOK_MAX_N), dtype=torch.int32, device=dev)
    toks = torch.empty(max(corpus_tokens.numel(), 1), dtype=torch.int32, device=dev)
    offs = torch.empty(doc_offsets.numel(), dtype=torch.int64, device=dev)
    n = C.c_int32(0)
    _check(lib.tasc_tok_enrich(_ptr(corpus_tokens), _ptr(doc_offsets), doc_offsets.numel() - 1, base_vocab, budget, n_max,
                               _ptr(merges), C.byref(n), _ptr(toks), _ptr(offs), _stream()), "tasc_tok_enrich")
    total = int(offs[-1].item())
    return merges[:n.value], toks[:total], offs


def tasc_tok_init_rows(matrix: torch.Tensor, merges: torch.Tensor) -> torch.Tensor:
    """Rows of the added tokens (mean of the constituents' rows) for an embedding / LM-head matrix [base_vocab, d]."""
    assert matrix.is_cuda and matrix.is_contiguous() and matrix.dtype in (torch.float32, torch.bfloat16)
    _dev(merges, torch.int32)
    base_vocab, d = matrix.shape
    rows = torch.zeros((merges.shape[0], d), dtype=matrix.dtype, device=matrix.device)
    status = torch.zeros(1, dtype=torch.int32, device=matrix.device)
    _check(lib.tasc_tok_init_rows(_ptr(matrix), F32 if matrix.dtype == torch.float32 else BF16, base_vocab, d, _ptr(merges),
                                  merges.shape[0], _ptr(rows), _ptr(status), _stream()), "tasc_tok_init_rows")
    code = int(status.item())
    if code != OK:
        raise TascError(code, "tasc_tok_init_rows (device)")
    return rows


def tasc_tok_encode(tokens: torch.Tensor, doc_offsets: torch.Tensor, base_vocab: int, merges: torch.Tensor):
    """Greedy longest-match encoding with the added tokens first.  Returns (tokens, offsets)."""
    _dev(tokens, torch.int32)
    _dev(doc_offsets, torch.int64)
    _dev(merges, torch.int32)
    dev = doc_offsets.device
    toks = torch.empty(max(tokens.numel(), 1), dtype=torch.int32, device=dev)
    offs = torch.empty(doc_offsets.numel(), dtype=torch.int64, device=dev)
    _check(lib.tasc_tok_encode(_ptr(tokens), _ptr(doc_offsets), doc_offsets.numel() - 1, base_vocab, _ptr(merges), merges.shape[0],
                               _ptr(toks), _ptr(offs), _stream()), "tasc_tok_encode")
    return toks[:int(offs[-1].item())], offs


def tasc_corpus_stats(corpus_tokens: torch.Tensor, doc_offsets: torch.Tensor, vocab: int, cdf_num: int = 4, cdf_den: int = 5) -> dict:
    """Corpus statistics as a dict with the field names of tasc_corpus_statistics."""
    _dev(corpus_tokens, torch.int32)
    _dev(doc_offsets, torch.int64)
    out = CorpusStatistics()
    _check(lib.tasc_corpus_stats(_ptr(corpus_tokens), _ptr(doc_offsets), doc_offsets.numel() - 1, vocab, cdf_num, cdf_den,
                                 _stream(), C.byref(out)), "tasc_corpus_stats")
    return {name: getattr(out, name) for name, _ in CorpusStatistics._fields_}


def tasc_draft(drafter: Drafter, tokens: torch.Tensor, length: torch.Tensor, k: int, lambda_num: int = 3,
               lambda_den: int = 4, out: torch.Tensor | None = None) -> torch.Tensor:
    _dev(tokens, torch.int32)
    _dev(length, torch.int32)
    B, stride = tokens.shape
    if out is None:
        out = torch.empty((B, k), dtype=torch.int32, device=tokens.device)
    _check(lib.tasc_draft(drafter._h, _ptr(tokens), stride, _ptr(length), B, k, lambda_num, lambda_den, _ptr(out), _stream()),
           "tasc_draft")
    return out


_TORCH_DTYPE = {F32: torch.float32, BF16: torch.bfloat16}


class Model:
    """tasc_model handle plus the device buffers it borrows (kept alive here)."""

    def __init__(self, shape, weights: dict, max_positions: int, page_size: int = 16):
        """``shape``: object with n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ff, vocab, dtype ("f32"/"bf16"),
        rope_base, rms_eps.  ``weights``: dict of CUDA tensors laid out as the C header describes."""
        self.shape = shape
        self.dtype = F32 if shape.dtype == "f32" else BF16
        self.tdtype = _TORCH_DTYPE[self.dtype]
        self.page_size = page_size
        self.max_positions = max_positions
        L = shape.n_layers
        self._keep = weights
        desc = ModelDesc(L, shape.d_model, shape.n_q_heads, shape.n_kv_heads, shape.head_dim, shape.d_ff, shape.vocab,
                         self.dtype, shape.rope_base, shape.rms_eps, max_positions, page_size)

        def arr(name, dtype):
            a = (C.c_void_p * L)()
            for l in range(L):
                a[l] = _dev(weights["layers"][l][name], dtype).data_ptr()
            return a

        self._arrays = [arr("attn_norm", torch.float32), arr("wqkv", self.tdtype), arr("wo", self.tdtype),
                        arr("mlp_norm", torch.float32), arr("w_gate_up", self.tdtype), arr("w_down", self.tdtype)]
        w = Weights(_dev(weights["embed"], self.tdtype).data_ptr(), _dev(weights["lm_head"], self.tdtype).data_ptr(),
                    _dev(weights["final_norm"], torch.float32).data_ptr(), *[C.cast(a, C.POINTER(C.c_void_p)) for a in self._arrays])
        h = _P()
        _check(lib.tasc_model_create(C.byref(desc), C.byref(w), C.byref(h)), "tasc_model_create")
        self._h = h

    def __del__(self):
        if getattr(self, "_h", None) and lib is not None:
            lib.tasc_model_destroy(self._h)
            self._h = None

    def workspace_bytes(self, B: int, k: int) -> int:
        n = lib.tasc_workspace_bytes(self._h, B, k)
        if n == 0:
            raise TascError(EINVAL, "tasc_workspace_bytes")
        return n

    def new_workspace(self, B: int, k: int, device="cuda") -> torch.Tensor:
        return torch.zeros(self.workspace_bytes(B, k), dtype=torch.uint8, device=device)

    def new_kv(self, B: int, max_len: int, device="cuda"):
        """A KV pool with one private run of pages per sequence: (pool, block_table, Kv struct)."""
        s = self.shape
        pages_per_seq = -(-max_len // self.page_size)
        n_pages = B * pages_per_seq
        pool = torch.zeros((s.n_layers, 2, n_pages, s.n_kv_heads, self.page_size, s.head_dim), dtype=self.tdtype, device=device)
        # pages of a sequence are deliberately not contiguous in the pool: page j of sequence b is j * B + b
        bt = (torch.arange(pages_per_seq, dtype=torch.int32)[None, :] * B + torch.arange(B, dtype=torch.int32)[:, None])
        bt = bt.contiguous().to(device)
        return pool, bt, Kv(pool.data_ptr(), n_pages, bt.data_ptr(), pages_per_seq)


def make_seqs(tokens: torch.Tensor, length: torch.Tensor, stop_len: torch.Tensor | None = None) -> Seqs:
    _dev(tokens, torch.int32)
    _dev(length, torch.int32)
    return Seqs(tokens.data_ptr(), tokens.shape[1], length.data_ptr(), None if stop_len is None else _dev(stop_len, torch.int32).data_ptr())


def tasc_prefill(model: Model, kv: Kv, seqs: Seqs, B: int, max_len: int, workspace: torch.Tensor):
    _check(lib.tasc_prefill(model._h, C.byref(kv), C.byref(seqs), B, max_len, _ptr(workspace), workspace.numel(), _stream()),
           "tasc_prefill")


def tasc_verify_step(model: Model, kv: Kv, seqs: Seqs, drafts: torch.Tensor, workspace: torch.Tensor, *,
                     forced_targets: torch.Tensor | None = None, want_targets: bool = False, want_logits: bool = False,
                     out: tuple | None = None):
    """Returns (n_accepted[B], next_token[B], target_tokens[B, k+1] or None, logits[B, k+1, V] or None).
    ``out``: caller-provided (n_accepted, next_token, target_tokens or None, logits or None) to write into."""
    _dev(drafts, torch.int32)
    B, k = drafts.shape
    dev = drafts.device
    if out is not None:
        n_acc, nxt, tgt, logits = out
        assert tuple(n_acc.shape) == (B,) and tuple(nxt.shape) == (B,)
        assert tgt is None or tuple(tgt.shape) == (B, k + 1)
        assert logits is None or tuple(logits.shape) == (B, k + 1, model.shape.vocab)
        for t, dt in ((n_acc, torch.int32), (nxt, torch.int32), (tgt, torch.int32), (logits, torch.float32)):
            if t is not None:
                _dev(t, dt)
    else:
        n_acc = torch.empty(B, dtype=torch.int32, device=dev)
        nxt = torch.empty(B, dtype=torch.int32, device=dev)
        tgt = torch.empty((B, k + 1), dtype=torch.int32, device=dev) if want_targets else None
        logits = torch.empty((B, k + 1, model.shape.vocab), dtype=torch.float32, device=dev) if want_logits else None
    if forced_targets is not None:
        _dev(forced_targets, torch.int32)
    _check(lib.tasc_verify_step(model._h, C.byref(kv), C.byref(seqs), _ptr(drafts), B, k, _ptr(forced_targets), _ptr(n_acc),
                                _ptr(nxt), _ptr(tgt), _ptr(logits), _ptr(workspace), workspace.numel(), _stream()),
           "tasc_verify_step")
    return n_acc, nxt, tgt, logits


def tasc_generate(model: Model, drafter: Drafter, kv: Kv, seqs: Seqs, B: int, max_new: int, k: int, workspace: torch.Tensor, *,
                  lambda_num: int = 3, lambda_den: int = 4, mode: int = MODE_GREEDY, forced_accept: int = 0,
                  continuation: torch.Tensor | None = None, out: torch.Tensor | None = None):
    """Returns (out[B, max_new] int32 CUDA tensor, Stats)."""
    if out is None:
        out = torch.empty((B, max_new), dtype=torch.int32, device=workspace.device)
    p = DraftParams(k, lambda_num, lambda_den, mode, forced_accept,
                    None if continuation is None else _dev(continuation, torch.int32).data_ptr(),
                    0 if continuation is None else continuation.shape[1])
    st = Stats()
    _check(lib.tasc_generate(model._h, drafter._h, C.byref(kv), C.byref(seqs), B, max_new, C.byref(p), _ptr(out), C.byref(st),
                             _ptr(workspace), workspace.numel(), _stream()), "tasc_generate")
    return out, st


def tasc_poll_status(workspace: torch.Tensor):
    _check(lib.tasc_poll_status(_ptr(workspace), _stream()), "tasc_poll_status")


def tasc_selftest_bounded_wait(workspace: torch.Tensor, budget_cycles: int = 200_000):
    """Launches the kernel that waits on a never-signalled barrier; tasc_poll_status(workspace) then raises ETIMEOUT."""
    _check(lib.tasc_selftest_bounded_wait(_ptr(workspace), budget_cycles, _stream()), "tasc_selftest_bounded_wait")


def tasc_gemm_bf16(x: torch.Tensor, w: torch.Tensor) -> torch.Tensor:
    """Y[M, N] float32 = X[M, K] @ W[N, K]^T for bf16 CUDA tensors."""
    _dev(x, torch.bfloat16)
    _dev(w, torch.bfloat16)
    M, K = x.shape
    N = w.shape[0]
    nbytes = lib.tasc_gemm_workspace_bytes(M, N, K)
    ws = torch.zeros(max(nbytes, 256), dtype=torch.uint8, device=x.device)
    y = torch.empty((M, N), dtype=torch.float32, device=x.device)
    _check(lib.tasc_gemm_bf16(_ptr(x), _ptr(w), _ptr(y), M, N, K, _ptr(ws), ws.numel(), _stream()), "tasc_gemm_bf16")
    tasc_poll_status(ws)
    return y


def tasc_gemm_bf16x2(x: torch.Tensor, w: torch.Tensor) -> torch.Tensor:
    """Y[M, N] float32 = X[M, K] @ W[N, K]^T for float32 X (carried as hi/lo bf16 pairs) and bf16 W."""
    _dev(x, torch.float32)
    _dev(w, torch.bfloat16)
    M, K = x.shape
    N = w.shape[0]
    ws = torch.zeros(max(lib.tasc_gemm_workspace_bytes(M, N, K), 256), dtype=torch.uint8, device=x.device)
    y = torch.empty((M, N), dtype=torch.float32, device=x.device)
    _check(lib.tasc_gemm_bf16x2(_ptr(x), _ptr(w), _ptr(y), M, N, K, _ptr(ws), ws.numel(), _stream()), "tasc_gemm_bf16x2")
    tasc_poll_status(ws)
    return y


def tasc_gemm_bf16_static(x: torch.Tensor, w: torch.Tensor, y: torch.Tensor, device_status: torch.Tensor | None = None):
    """Y[M, N] float32 = X[M, K] @ W[N, K]^T for bf16 CUDA tensors, written into the caller's ``y``.

    For callers that cannot allocate device memory: the split-K partial sums use the library's fixed
    8 MiB device array, so this wrapper (unlike ``tasc_gemm_bf16``) creates no tensor either.
    ``device_status``: optional int32[1] CUDA tensor that receives a device-side error code.  Raises
    TascError(ECAPACITY) when M * N * 4 bytes exceed the array."""
    _dev(x, torch.bfloat16)
    _dev(w, torch.bfloat16)
    _dev(y, torch.float32)
    M, K = x.shape
    N = w.shape[0]
    assert tuple(y.shape) == (M, N)
    if device_status is not None:
        _dev(device_status, torch.int32)
    _check(lib.tasc_gemm_bf16_static(_ptr(x), _ptr(w), _ptr(y), M, N, K, _ptr(device_status), _stream()),
           "tasc_gemm_bf16_static")
    return y


def weights_to_device(w: dict, dtype: str, device="cuda") -> dict:
    """Host float32 weight dict (as produced by the workload generator) -> CUDA tensors in the model dtype."""
    td = torch.float32 if dtype == "f32" else torch.bfloat16
    conv = lambda a, t: torch.from_numpy(np.ascontiguousarray(a)).to(device=device, dtype=t).contiguous()
    out = {"embed": conv(w["embed"], td), "final_norm": conv(w["final_norm"], torch.float32), "layers": []}
    out["lm_head"] = out["embed"] if w["lm_head"] is w["embed"] else conv(w["lm_head"], td)
    for lw in w["layers"]:
        out["layers"].append({k: conv(v, torch.float32 if k.endswith("norm") else td) for k, v in lw.items()})
    return out


def profile_kinds():
    return [lib.tasc_profile_kind_name(i).decode() for i in range(lib.tasc_profile_kinds())]


def tasc_profile_enable(on: bool):
    _check(lib.tasc_profile_enable(1 if on else 0), "tasc_profile_enable")


def tasc_profile_read() -> dict:
    """{kind: (milliseconds, timed launches)} since the last read."""
    n = lib.tasc_profile_kinds()
    ms = (C.c_double * n)()
    cnt = (C.c_int64 * n)()
    _check(lib.tasc_profile_read(ms, cnt, n), "tasc_profile_read")
    return {k: (ms[i], cnt[i]) for i, k in enumerate(profile_kinds())}


def tasc_launch_counts() -> dict:
    n = lib.tasc_profile_kinds()
    cnt = (C.c_int64 * n)()
    _check(lib.tasc_launch_counts(cnt, n), "tasc_launch_counts")
    return {k: cnt[i] for i, k in enumerate(profile_kinds())}
