"""ctypes binding of libspecvla.so: argument marshalling only.

PyTorch is used for device memory (weights, workspace, inputs) and the current stream;
all computation happens inside the library. Method names follow the C entry points.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

from .build import LIB_PATH

MAX_DEPTH = 8
MAX_TREE_ROWS = 128

OPT_PERSISTENT_FORWARD, OPT_DEPENDENT_LAUNCH, OPT_L2_PREFETCH, OPT_WAIT_LIMIT_NS, OPT_DEVICE_LOOP = 1, 2, 3, 4, 5
BUF_GREEDY, BUF_MARGIN, BUF_FEATURES, BUF_PATH, BUF_STATE, BUF_TOPK_TOK, BUF_TOPK_LP = 1, 2, 3, 4, 5, 6, 7


class ModelDesc(C.Structure):
    _fields_ = [(n, C.c_int) for n in ("n_layers", "d_model", "n_heads", "head_dim", "d_ffn", "vocab",
                                       "action_base", "n_bins")] + \
               [("rms_eps", C.c_float), ("rope_theta", C.c_float)] + \
               [(n, C.c_int) for n in ("max_seq", "max_episodes", "max_rows", "action_only", "weight_bits")]


class Weights(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("lm_head", C.c_void_p), ("final_norm", C.c_void_p)] + \
               [(n, C.POINTER(C.c_void_p)) for n in ("wqkv", "wo", "wgu", "wd", "norm1", "norm2")]


class DraftWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("fc", "wqkv", "wo", "wgu", "wd", "norm1", "norm2")]


class TreeShape(C.Structure):
    _fields_ = [("depth", C.c_int), ("branch", C.c_int * MAX_DEPTH), ("expand", C.c_int * MAX_DEPTH),
                ("prune", C.c_int), ("keep", C.c_int)]


class Tree(C.Structure):
    _fields_ = [("n_rows", C.c_int), ("tokens", C.POINTER(C.c_int)), ("parent", C.POINTER(C.c_int)),
                ("depth", C.POINTER(C.c_int)), ("score", C.POINTER(C.c_float))]


class Stats(C.Structure):
    _fields_ = [("iterations", C.c_int), ("tokens_emitted", C.c_int), ("accept_len", C.c_int * 16),
                ("ms_prefill", C.c_float), ("ms_draft", C.c_float), ("ms_verify", C.c_float),
                ("pos_iterations", C.c_int * 16), ("pos_accept_sum", C.c_int * 16),
                ("ms_loop", C.c_float), ("device_loop", C.c_int)]


EXPORTS = {
    "specvla_workspace_bytes": (C.c_size_t, [C.POINTER(ModelDesc)]),
    "specvla_create": (C.c_int, [C.POINTER(ModelDesc), C.POINTER(Weights), C.POINTER(DraftWeights),
                                 C.c_void_p, C.c_size_t, C.POINTER(C.c_void_p)]),
    "specvla_destroy": (C.c_int, [C.c_void_p]),
    "specvla_reset": (C.c_int, [C.c_void_p, C.c_int]),
    "specvla_set_option": (C.c_int, [C.c_void_p, C.c_int, C.c_longlong]),
    "specvla_prefill": (C.c_int, [C.c_void_p, C.c_int, C.POINTER(C.c_int), C.c_void_p, C.POINTER(C.c_int),
                                  C.POINTER(C.c_int), C.POINTER(C.c_int), C.c_void_p, C.c_void_p]),
    "specvla_draft_tree": (C.c_int, [C.c_void_p, C.c_int, C.POINTER(C.c_int), C.POINTER(TreeShape),
                                     C.POINTER(Tree), C.c_void_p]),
    "specvla_verify_tree": (C.c_int, [C.c_void_p, C.c_int, C.POINTER(C.c_int), C.POINTER(Tree), C.c_int,
                                      C.POINTER(C.c_int), C.POINTER(C.c_int), C.c_void_p, C.c_void_p]),
    "specvla_score_tree": (C.c_int, [C.c_void_p, C.c_int, C.POINTER(C.c_int), C.POINTER(Tree), C.POINTER(C.c_int),
                                     C.c_void_p]),
    "specvla_generate_action": (C.c_int, [C.c_void_p, C.c_int, C.POINTER(C.c_int), C.c_void_p,
                                          C.POINTER(C.c_int), C.POINTER(C.c_int), C.POINTER(TreeShape),
                                          C.c_int, C.c_int, C.POINTER(C.c_int), C.POINTER(C.c_float),
                                          C.POINTER(Stats), C.c_void_p]),
    "specvla_read_buffer": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p, C.c_size_t, C.c_void_p]),
    "specvla_read_kv": (C.c_int, [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int,
                                  C.c_void_p, C.c_void_p]),
    "specvla_gemm_scratch_bytes": (C.c_size_t, [C.c_int, C.c_int, C.c_int]),
    "specvla_gemm": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int,
                                    C.c_void_p, C.c_size_t, C.c_void_p]),
    "specvla_gemm_status": (C.c_int, [C.c_void_p, C.c_void_p]),
    "specvla_packed_weight_bytes": (C.c_size_t, [C.c_int, C.c_int]),
    "specvla_pack_weights": (C.c_int, [C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_size_t, C.c_void_p]),
    "specvla_gemm_prepacked": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int,
                                         C.c_void_p, C.c_size_t, C.c_void_p]),
    "specvla_gemm_fault_test": (C.c_int, [C.c_longlong, C.c_int]),
    "specvla_gemm_static_status": (C.c_int, [C.c_void_p]),
    "specvla_gemm_static": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int,
                                     C.c_void_p]),
    "specvla_profile": (C.c_int, [C.c_void_p, C.c_int]),
    "specvla_profile_read": (C.c_int, [C.c_void_p, C.POINTER(C.c_double), C.POINTER(C.c_longlong),
                                       C.POINTER(C.c_double)]),
    "specvla_strerror": (C.c_char_p, [C.c_int]),
    "specvla_last_cuda_error": (C.c_char_p, [C.c_void_p]),
    "specvla_kernel_launches": (C.c_longlong, [C.c_void_p]),
}


def load_library(path: str = LIB_PATH) -> C.CDLL:
    if not os.path.exists(path):
        raise RuntimeError(f"{path} is missing: build it with `python -m paper_2507_22424_b200.build` "
                           "(there is no fallback implementation)")
    lib = C.CDLL(path)
    for name, (res, args) in EXPORTS.items():
        fn = getattr(lib, name)
        fn.restype, fn.argtypes = res, args
    return lib


lib = load_library()


class SpecVLAError(RuntimeError):
    def __init__(self, code, detail=""):
        self.code = code
        super().__init__(f"specvla error {code}: {lib.specvla_strerror(code).decode()} {detail}")


def _ints(values):
    return (C.c_int * len(values))(*[int(v) for v in values])


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def make_shape(branch, expand, prune: bool = False, keep: int = 0) -> TreeShape:
    s = TreeShape()
    s.depth = len(branch)
    s.prune = 1 if prune else 0
    s.keep = int(keep)
    for i, (b, e) in enumerate(zip(branch, expand)):
        s.branch[i], s.expand[i] = int(b), int(e)
    return s


class SpecVLA:
    """One library context over weights held in torch CUDA tensors (kept alive here)."""

    def __init__(self, desc, weights: dict, max_seq=512, max_episodes=1, max_rows=512, action_only=True,
                 weight_bits=16):
        self.model = desc
        self.md = ModelDesc(desc.n_layers, desc.d_model, desc.n_heads, desc.head_dim, desc.d_ffn, desc.vocab,
                            desc.action_base, desc.n_bins, desc.rms_eps, desc.rope_theta,
                            max_seq, max_episodes, max_rows, int(action_only), int(weight_bits))
        self.w = weights
        L = desc.n_layers

        def per_layer(name):
            return (C.c_void_p * L)(*[weights[f"layers.{l}.{name}"].data_ptr() for l in range(L)])

        self._arrays = {n: per_layer(n) for n in ("wqkv", "wo", "wgu", "wd", "norm1", "norm2")}
        tw = Weights(weights["embed"].data_ptr(), weights["lm_head"].data_ptr(),
                     weights["final_norm"].data_ptr(), *[self._arrays[n] for n in
                                                         ("wqkv", "wo", "wgu", "wd", "norm1", "norm2")])
        dw = None
        if "draft.fc" in weights:
            dw = DraftWeights(weights["draft.fc"].data_ptr(),
                              *[weights[f"draft.layer.{n}"].data_ptr()
                                for n in ("wqkv", "wo", "wgu", "wd", "norm1", "norm2")])
        nbytes = lib.specvla_workspace_bytes(C.byref(self.md))
        if nbytes == 0:
            raise SpecVLAError(-1, "(model description rejected)")
        self.workspace = torch.empty(nbytes + 1024, dtype=torch.uint8, device="cuda")
        base = (self.workspace.data_ptr() + 1023) // 1024 * 1024
        self.workspace_bytes = nbytes
        handle = C.c_void_p()
        rc = lib.specvla_create(C.byref(self.md), C.byref(tw), C.byref(dw) if dw else None,
                                C.c_void_p(base), nbytes, C.byref(handle))
        if rc != 0:
            raise SpecVLAError(rc)
        self.h = handle

    def close(self):
        if getattr(self, "h", None):
            lib.specvla_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_option(self, option: int, value: int):
        self._check(lib.specvla_set_option(self.h, int(option), int(value)))

    def _check(self, rc):
        if rc != 0:
            raise SpecVLAError(rc, lib.specvla_last_cuda_error(self.h).decode())

    # ------------------------------------------------------------------ entry points
    def prefill(self, episodes, embeds, token_ids, lens, want_logits=False):
        """embeds: CUDA bf16 [sum(lens), d]; token_ids: host ints; returns first tokens."""
        n = len(episodes)
        first = (C.c_int * n)()
        logits = torch.empty(n, self.model.vocab, dtype=torch.float32, device="cuda") if want_logits else None
        self._check(lib.specvla_prefill(self.h, n, _ints(episodes), C.c_void_p(embeds.data_ptr()),
                                        _ints(token_ids), _ints(lens), first,
                                        C.c_void_p(logits.data_ptr()) if want_logits else None, _stream()))
        return (list(first), logits) if want_logits else list(first)

    def draft_tree(self, episodes, shape: TreeShape, want_trees=True):
        n = len(episodes)
        if not want_trees:
            self._check(lib.specvla_draft_tree(self.h, n, _ints(episodes), C.byref(shape), None, _stream()))
            return None
        trees = (Tree * n)()
        bufs = []
        for i in range(n):
            b = [(C.c_int * MAX_TREE_ROWS)() for _ in range(3)] + [(C.c_float * MAX_TREE_ROWS)()]
            bufs.append(b)
            trees[i].tokens, trees[i].parent, trees[i].depth = b[0], b[1], b[2]
            trees[i].score = b[3]
        self._check(lib.specvla_draft_tree(self.h, n, _ints(episodes), C.byref(shape), trees, _stream()))
        out = []
        for i in range(n):
            k = trees[i].n_rows
            out.append(dict(tokens=list(bufs[i][0][:k]), parent=list(bufs[i][1][:k]),
                            depth=list(bufs[i][2][:k]), score=list(bufs[i][3][:k])))
        return out

    def verify_tree(self, episodes, trees, r, want_logits=False):
        """trees: list of dicts (tokens, parent, depth) or None for the device-resident trees.
        Returns (accept lengths, emitted tokens per episode[, logits [rows, V]])."""
        n = len(episodes)
        ctrees, keep, rows = None, [], 0
        if trees is not None:
            ctrees = (Tree * n)()
            for i, t in enumerate(trees):
                a, b, c = _ints(t["tokens"]), _ints(t["parent"]), _ints(t["depth"])
                keep += [a, b, c]
                ctrees[i].n_rows = len(t["tokens"])
                ctrees[i].tokens, ctrees[i].parent, ctrees[i].depth = a, b, c
                ctrees[i].score = None
                rows += len(t["tokens"])
        logits = None
        if want_logits:
            if trees is None:
                raise ValueError("want_logits needs caller-supplied trees (row count)")
            logits = torch.empty(rows, self.model.vocab, dtype=torch.float32, device="cuda")
        m = (C.c_int * n)()
        toks = (C.c_int * (n * (MAX_DEPTH + 1)))()
        self._check(lib.specvla_verify_tree(self.h, n, _ints(episodes), ctrees, int(r), m, toks,
                                            C.c_void_p(logits.data_ptr()) if want_logits else None, _stream()))
        emitted = [list(toks[i * (MAX_DEPTH + 1): i * (MAX_DEPTH + 1) + m[i] + 1]) for i in range(n)]
        return (list(m), emitted, logits) if want_logits else (list(m), emitted)

    def score_tree(self, episodes, trees):
        """Greedy token of the target after every row of the given trees; episode state untouched."""
        n = len(episodes)
        ctrees, keep, rows = (Tree * n)(), [], 0
        for i, t in enumerate(trees):
            a, b, c = _ints(t["tokens"]), _ints(t["parent"]), _ints(t["depth"])
            keep += [a, b, c]
            ctrees[i].n_rows = len(t["tokens"])
            ctrees[i].tokens, ctrees[i].parent, ctrees[i].depth = a, b, c
            ctrees[i].score = None
            rows += len(t["tokens"])
        g = (C.c_int * rows)()
        self._check(lib.specvla_score_tree(self.h, n, _ints(episodes), ctrees, g, _stream()))
        return list(g)

    def generate_action(self, episodes, embeds, token_ids, lens, shape: TreeShape, r, n_tokens=7):
        n = len(episodes)
        toks = (C.c_int * (n * n_tokens))()
        acts = (C.c_float * (n * n_tokens))()
        stats = Stats()
        self._check(lib.specvla_generate_action(self.h, n, _ints(episodes), C.c_void_p(embeds.data_ptr()),
                                                _ints(token_ids), _ints(lens), C.byref(shape), int(r),
                                                int(n_tokens), toks, acts, C.byref(stats), _stream()))
        tokens = [list(toks[i * n_tokens:(i + 1) * n_tokens]) for i in range(n)]
        actions = [list(acts[i * n_tokens:(i + 1) * n_tokens]) for i in range(n)]
        return tokens, actions, stats

    # ------------------------------------------------------------------ inspection
    def read_buffer(self, what, count, dtype):
        out = torch.empty(count, dtype=dtype)
        self._check(lib.specvla_read_buffer(self.h, what, C.c_void_p(out.data_ptr()),
                                            out.numel() * out.element_size(), _stream()))
        return out

    def read_kv(self, episode, layer, which, slot0, n_slots, draft=False):
        hd = self.model.n_heads * self.model.head_dim
        out = torch.empty(n_slots, hd, dtype=torch.float32)
        self._check(lib.specvla_read_kv(self.h, int(draft), episode, layer, which, slot0, n_slots,
                                        C.c_void_p(out.data_ptr()), _stream()))
        return out

    def profile(self, enable: bool):
        self._check(lib.specvla_profile(self.h, int(enable)))

    def profile_read(self):
        """Per weight-matrix class: (ms, launches, weight bytes) summed since profiling was enabled."""
        ms, n, by = (C.c_double * 6)(), (C.c_longlong * 6)(), (C.c_double * 6)()
        self._check(lib.specvla_profile_read(self.h, ms, n, by))
        names = ("qkv", "o", "gate_up", "down", "lm_head", "fc")
        return {k: dict(ms=ms[i], launches=int(n[i]), bytes=by[i]) for i, k in enumerate(names)}

    def kernel_launches(self):
        return int(lib.specvla_kernel_launches(self.h))


def gemm(x: torch.Tensor, w: torch.Tensor) -> torch.Tensor:
    """Y[T, N] = X[T, K] (f32) @ W[N, K]^T (bf16) through the library's weight-streaming GEMM."""
    assert x.dtype == torch.float32 and w.dtype == torch.bfloat16
    T, K = x.shape
    N = w.shape[0]
    y = torch.empty(T, N, dtype=torch.float32, device="cuda")
    nb = lib.specvla_gemm_scratch_bytes(T, N, K)
    scratch = torch.empty(nb + 1024, dtype=torch.uint8, device="cuda")
    sp = (scratch.data_ptr() + 1023) // 1024 * 1024
    rc = lib.specvla_gemm(C.c_void_p(x.data_ptr()), C.c_void_p(w.data_ptr()), C.c_void_p(y.data_ptr()),
                               T, N, K, C.c_void_p(sp), nb, _stream())
    if rc == 0:
        rc = lib.specvla_gemm_status(C.c_void_p(sp), _stream())
    if rc != 0:
        raise SpecVLAError(rc)
    return y


def pack_weights(w: torch.Tensor) -> torch.Tensor:
    """The library's streaming form of W [N, K] (bf16): specvla_pack_weights into a new buffer."""
    assert w.dtype == torch.bfloat16 and w.is_contiguous()
    N, K = w.shape
    nb = lib.specvla_packed_weight_bytes(N, K)
    if nb == 0:
        raise SpecVLAError(-1, "(shape rejected)")
    buf = torch.empty(nb + 1024, dtype=torch.uint8, device="cuda")
    off = (-buf.data_ptr()) % 1024
    packed = buf[off:off + nb]
    rc = lib.specvla_pack_weights(C.c_void_p(w.data_ptr()), N, K, C.c_void_p(packed.data_ptr()), nb, _stream())
    if rc != 0:
        raise SpecVLAError(rc)
    return packed


def gemm_prepacked(x: torch.Tensor, packed: torch.Tensor, N: int) -> torch.Tensor:
    """Y[T, N] = X[T, K] (f32) @ W^T with W given in packed form (pack_weights)."""
    T, K = x.shape
    y = torch.empty(T, N, dtype=torch.float32, device="cuda")
    nb = lib.specvla_gemm_scratch_bytes(T, N, K)
    scratch = torch.empty(nb + 1024, dtype=torch.uint8, device="cuda")
    sp = (scratch.data_ptr() + 1023) // 1024 * 1024
    rc = lib.specvla_gemm_prepacked(C.c_void_p(x.data_ptr()), C.c_void_p(packed.data_ptr()), C.c_void_p(y.data_ptr()),
                                    T, N, K, C.c_void_p(sp), nb, _stream())
    if rc == 0:
        rc = lib.specvla_gemm_status(C.c_void_p(sp), _stream())
    if rc != 0:
        raise SpecVLAError(rc)
    return y


STATIC_SCRATCH_BYTES = 16 << 20


def gemm_static(x: torch.Tensor, w: torch.Tensor, y: torch.Tensor) -> torch.Tensor:
    """specvla_gemm_static: the same product written into the caller's y, with the scratch taken
    from the library's built-in array instead of a caller allocation. Nothing is allocated here
    or in the library; shapes whose scratch exceeds STATIC_SCRATCH_BYTES raise SpecVLAError(-2)."""
    assert x.dtype == torch.float32 and w.dtype == torch.bfloat16 and y.dtype == torch.float32
    T, K = x.shape
    N = w.shape[0]
    assert y.shape == (T, N) and y.is_contiguous()
    rc = lib.specvla_gemm_static(C.c_void_p(x.data_ptr()), C.c_void_p(w.data_ptr()), C.c_void_p(y.data_ptr()),
                                 T, N, K, 1, _stream())
    if rc != 0:
        raise SpecVLAError(rc)
    return y


class GemmRunner:
    """specvla_gemm with output and scratch allocated once (for timing loops)."""

    def __init__(self, T: int, N: int, K: int):
        self.T, self.N, self.K = T, N, K
        self.y = torch.empty(T, N, dtype=torch.float32, device="cuda")
        self.nb = lib.specvla_gemm_scratch_bytes(T, N, K)
        self.scratch = torch.empty(self.nb + 1024, dtype=torch.uint8, device="cuda")
        self.sp = (self.scratch.data_ptr() + 1023) // 1024 * 1024

    def __call__(self, x: torch.Tensor, w: torch.Tensor) -> torch.Tensor:
        rc = lib.specvla_gemm(C.c_void_p(x.data_ptr()), C.c_void_p(w.data_ptr()), C.c_void_p(self.y.data_ptr()),
                              self.T, self.N, self.K, C.c_void_p(self.sp), self.nb, _stream())
        if rc != 0:
            raise SpecVLAError(rc)
        return self.y
