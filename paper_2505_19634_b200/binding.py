"""ctypes binding of libtts_b200.so.  Argument marshalling only.

Device arrays are passed as torch CUDA tensors (or raw integer addresses); torch is used for
device memory and streams and nothing else.  There is no fallback: if the shared library is
missing, loading raises.
"""
from __future__ import annotations

import ctypes
from ctypes import POINTER, byref, c_char_p, c_double, c_float, c_int, c_int32, c_int64, c_void_p
from pathlib import Path
from typing import Optional, Sequence

_PKG = Path(__file__).resolve().parent
_LIB_PATH = _PKG / "libtts_b200.so"

MASK_CAUSAL, MASK_TREE = 0, 1
OUT_BF16, OUT_FP32 = 0, 1
LOGITS_BF16, LOGITS_FP32 = 0, 1
ATTN_AUTO, ATTN_SIMT, ATTN_TCGEN05, ATTN_TCGEN05_TOKEN_MAJOR, ATTN_TCGEN05_ROW_MAJOR = 0, 1, 2, 3, 4

EXPORTED_SYMBOLS = (
    "tts_create", "tts_destroy", "tts_set_stream", "tts_verify_attn", "tts_verify_attn_tree", "tts_attn_plan",
    "tts_attn_plan_drop", "tts_verify_attn_groups", "tts_attn_plan_groups",
    "tts_accept", "tts_accept_logits", "tts_verify_step_host_logits", "tts_majority_vote", "tts_confidence_max", "tts_greedy_search", "tts_grid_search", "tts_last_status",
    "tts_last_cuda_error", "tts_launch_count", "tts_strerror", "tts_verify_step_host",
    "tts_profile_enable", "tts_profile_read", "tts_debug_wait_timeout", "tts_verify_attn_noalloc", "tts_kv_append", "tts_kv_rollback", "tts_accept_tree",
)


class TtsError(RuntimeError):
    def __init__(self, status: int, where: str, cuda_error: int = 0):
        self.status = status
        self.cuda_error = cuda_error
        extra = f" (cudaError {cuda_error})" if cuda_error else ""
        super().__init__(f"{where}: {tts_strerror(status)} [{status}]{extra}")


class TtsConfig(ctypes.Structure):
    _fields_ = [("n_q_heads", c_int32), ("n_kv_heads", c_int32), ("head_dim", c_int32),
                ("page_size", c_int32), ("max_branches", c_int32), ("max_rows_per_branch", c_int32),
                ("max_blocks_per_branch", c_int32), ("num_pages", c_int32), ("out_dtype", c_int32),
                ("attn_impl", c_int32), ("softmax_scale", c_float), ("debug_bounds", c_int32),
                ("max_ctas", c_int32)]


class TtsSearchLimits(ctypes.Structure):
    _fields_ = [("max_branches", c_int32), ("max_gamma", c_int32), ("max_steps", c_int32)]


_TASK_FN = ctypes.CFUNCTYPE(c_double, c_int, c_int, c_void_p)
_lib: Optional[ctypes.CDLL] = None


def library_path() -> Path:
    return _LIB_PATH


def load_library() -> ctypes.CDLL:
    """Loads the in-tree shared library; raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not _LIB_PATH.exists():
        raise FileNotFoundError(
            f"{_LIB_PATH} is missing: build it with `python -m paper_2505_19634_b200.build` "
            "(there is no fallback implementation)")
    lib = ctypes.CDLL(str(_LIB_PATH))
    vp, ip = c_void_p, POINTER(c_int32)
    lib.tts_create.argtypes = [POINTER(TtsConfig), POINTER(c_void_p)]
    lib.tts_destroy.argtypes = [vp]
    lib.tts_set_stream.argtypes = [vp, vp]
    lib.tts_verify_attn.argtypes = [vp, vp, vp, vp, vp, c_int, vp, c_int, c_int, c_int, vp]
    lib.tts_verify_attn_tree.argtypes = [vp, vp, vp, vp, vp, c_int, vp, vp, c_int, c_int, vp]
    lib.tts_attn_plan.argtypes = [vp, vp, c_int, vp, c_int, c_int]
    lib.tts_attn_plan_drop.argtypes = [vp]
    lib.tts_verify_attn_groups.argtypes = [vp, vp, vp, vp, vp, ip, ip, c_int, vp, c_int, c_int, vp]
    lib.tts_attn_plan_groups.argtypes = [vp, vp, ip, ip, c_int, vp, c_int, c_int]
    lib.tts_accept.argtypes = [vp, vp, vp, vp, vp, c_int, c_int, c_int, vp, vp]
    lib.tts_accept_logits.argtypes = [vp, vp, vp, c_int, vp, vp, c_int, c_int, c_int, vp, vp]
    lib.tts_verify_step_host_logits.argtypes = [vp, c_int, vp, POINTER(c_void_p), POINTER(c_void_p), vp, c_int, vp,
                                                c_int, c_int, vp, vp, c_int, vp, vp, c_int, vp, vp, vp]
    lib.tts_accept_tree.argtypes = [vp, vp, vp, vp, vp, vp, c_int, c_int, c_int, vp, vp, vp]
    lib.tts_kv_append.argtypes = [vp, vp, vp, vp, vp, vp, c_int, vp, c_int, c_int]
    lib.tts_kv_rollback.argtypes = [vp, vp, vp, c_int, c_int]
    lib.tts_majority_vote.argtypes = [POINTER(c_int64), POINTER(c_float), c_int, POINTER(c_int64), POINTER(c_int)]
    lib.tts_confidence_max.argtypes = lib.tts_majority_vote.argtypes
    lib.tts_greedy_search.argtypes = [_TASK_FN, vp, POINTER(TtsSearchLimits), POINTER(c_int), POINTER(c_int),
                                      POINTER(c_double), POINTER(c_int), POINTER(c_int)]
    lib.tts_grid_search.argtypes = [_TASK_FN, vp, POINTER(TtsSearchLimits), POINTER(c_int), POINTER(c_int),
                                    POINTER(c_double), POINTER(c_int)]
    lib.tts_last_status.argtypes = [vp, POINTER(c_int)]
    lib.tts_last_cuda_error.argtypes = [vp]
    lib.tts_launch_count.argtypes = [vp]
    lib.tts_launch_count.restype = c_int64
    lib.tts_debug_wait_timeout.argtypes = [vp, c_int64]
    lib.tts_profile_enable.argtypes = [vp, c_int]
    lib.tts_profile_read.argtypes = [vp, POINTER(c_float), POINTER(c_float), POINTER(c_int)]
    lib.tts_strerror.argtypes = [c_int]
    lib.tts_strerror.restype = c_char_p
    lib.tts_verify_step_host.argtypes = [vp, c_int, vp, POINTER(c_void_p), POINTER(c_void_p), vp, c_int, vp,
                                         c_int, c_int, vp, vp, vp, vp, c_int, vp, vp, vp]
    lib.tts_verify_attn_noalloc.argtypes = [vp, vp, vp, vp, c_int, c_int, vp, c_int, c_int, c_int, c_int, vp, vp]
    for name in EXPORTED_SYMBOLS:
        fn = getattr(lib, name)
        if name not in ("tts_launch_count", "tts_strerror"):
            fn.restype = c_int
    _lib = lib
    return lib


def tts_strerror(status: int) -> str:
    try:
        return load_library().tts_strerror(int(status)).decode()
    except FileNotFoundError:
        return f"status {status}"


def _ptr(x) -> c_void_p:
    """Address of a torch tensor / numpy array / int / None."""
    if x is None:
        return c_void_p(0)
    if isinstance(x, int):
        return c_void_p(x)
    if hasattr(x, "data_ptr"):
        return c_void_p(x.data_ptr())
    if hasattr(x, "ctypes"):
        return c_void_p(x.ctypes.data)
    raise TypeError(f"cannot take the address of {type(x)}")


class TtsContext:
    """Owns one tts_ctx on the current CUDA device.  Methods mirror the C-ABI names."""

    def __init__(self, n_q_heads: int, n_kv_heads: int, max_branches: int, max_rows_per_branch: int,
                 max_blocks_per_branch: int, num_pages: int, out_dtype: int = OUT_BF16,
                 attn_impl: int = ATTN_AUTO, softmax_scale: float = 0.0, debug_bounds: bool = False,
                 head_dim: int = 128, page_size: int = 16, stream=None, max_ctas: int = 0):
        self._lib = load_library()
        self.cfg = TtsConfig(n_q_heads, n_kv_heads, head_dim, page_size, max_branches, max_rows_per_branch,
                             max_blocks_per_branch, num_pages, out_dtype, attn_impl, softmax_scale,
                             1 if debug_bounds else 0, int(max_ctas))
        self._h = c_void_p(0)
        rc = self._lib.tts_create(byref(self.cfg), byref(self._h))
        if rc != 0:
            self._h = c_void_p(0)
            raise TtsError(rc, "tts_create")
        if stream is not None:
            self.tts_set_stream(stream)

    # -- lifetime ---------------------------------------------------------------------------
    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value:
            self._lib.tts_destroy(self._h)
            self._h = c_void_p(0)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    def _check(self, rc: int, where: str):
        if rc != 0:
            raise TtsError(rc, where, self._lib.tts_last_cuda_error(self._h) if rc == -3 else 0)

    # -- C-ABI mirrors ----------------------------------------------------------------------
    def tts_set_stream(self, stream):
        handle = stream if isinstance(stream, int) or stream is None else stream.cuda_stream
        self._check(self._lib.tts_set_stream(self._h, c_void_p(handle or 0)), "tts_set_stream")

    def tts_verify_attn(self, q, k_pages, v_pages, block_table, prefix_len: int, branch_lens,
                        n_branches: int, gamma: int, mask_kind: int, out):
        self._check(self._lib.tts_verify_attn(self._h, _ptr(q), _ptr(k_pages), _ptr(v_pages), _ptr(block_table),
                                              int(prefix_len), _ptr(branch_lens), int(n_branches), int(gamma),
                                              int(mask_kind), _ptr(out)), "tts_verify_attn")

    def tts_attn_plan(self, block_table, prefix_len: int, branch_lens, n_branches: int, rows_per_branch: int):
        self._check(self._lib.tts_attn_plan(self._h, _ptr(block_table), int(prefix_len), _ptr(branch_lens),
                                            int(n_branches), int(rows_per_branch)), "tts_attn_plan")

    @staticmethod
    def _host_i32(values):
        return (c_int32 * len(values))(*[int(v) for v in values])

    def tts_verify_attn_groups(self, q, k_pages, v_pages, block_table, group_sizes, group_prefix_len, branch_lens,
                               n_branches: int, gamma: int, out):
        """group_sizes and group_prefix_len are host sequences of equal length."""
        self._check(self._lib.tts_verify_attn_groups(self._h, _ptr(q), _ptr(k_pages), _ptr(v_pages), _ptr(block_table),
                                                     self._host_i32(group_sizes), self._host_i32(group_prefix_len),
                                                     len(group_sizes), _ptr(branch_lens), int(n_branches), int(gamma),
                                                     _ptr(out)), "tts_verify_attn_groups")

    def tts_attn_plan_groups(self, block_table, group_sizes, group_prefix_len, branch_lens, n_branches: int,
                             rows_per_branch: int):
        self._check(self._lib.tts_attn_plan_groups(self._h, _ptr(block_table), self._host_i32(group_sizes),
                                                   self._host_i32(group_prefix_len), len(group_sizes), _ptr(branch_lens),
                                                   int(n_branches), int(rows_per_branch)), "tts_attn_plan_groups")

    def tts_attn_plan_drop(self):
        self._check(self._lib.tts_attn_plan_drop(self._h), "tts_attn_plan_drop")

    def tts_verify_attn_tree(self, q, k_pages, v_pages, block_table, prefix_len: int, branch_lens,
                             tree_parents, n_branches: int, n_nodes: int, out):
        self._check(self._lib.tts_verify_attn_tree(self._h, _ptr(q), _ptr(k_pages), _ptr(v_pages),
                                                   _ptr(block_table), int(prefix_len), _ptr(branch_lens),
                                                   _ptr(tree_parents), int(n_branches), int(n_nodes), _ptr(out)),
                    "tts_verify_attn_tree")

    def tts_accept(self, p_target, q_draft, draft_tokens, uniforms, n_branches: int, gamma: int, vocab: int,
                   accepted_len, next_token):
        self._check(self._lib.tts_accept(self._h, _ptr(p_target), _ptr(q_draft), _ptr(draft_tokens), _ptr(uniforms),
                                         int(n_branches), int(gamma), int(vocab), _ptr(accepted_len),
                                         _ptr(next_token)), "tts_accept")

    def tts_accept_logits(self, target_logits, draft_logits, logits_dtype: int, draft_tokens, uniforms,
                          n_branches: int, gamma: int, vocab: int, accepted_len, next_token):
        self._check(self._lib.tts_accept_logits(self._h, _ptr(target_logits), _ptr(draft_logits), int(logits_dtype),
                                                _ptr(draft_tokens), _ptr(uniforms), int(n_branches), int(gamma),
                                                int(vocab), _ptr(accepted_len), _ptr(next_token)), "tts_accept_logits")

    def tts_accept_tree(self, p_target, q_draft, draft_tokens, tree_parents, uniforms, n_branches: int, n_nodes: int,
                        vocab: int, accepted_len, last_node, next_token):
        self._check(self._lib.tts_accept_tree(self._h, _ptr(p_target), _ptr(q_draft), _ptr(draft_tokens),
                                              _ptr(tree_parents), _ptr(uniforms), int(n_branches), int(n_nodes),
                                              int(vocab), _ptr(accepted_len), _ptr(last_node), _ptr(next_token)),
                    "tts_accept_tree")

    def tts_kv_append(self, k_new, v_new, k_pages, v_pages, block_table, prefix_len: int, branch_lens,
                      n_branches: int, rows: int):
        self._check(self._lib.tts_kv_append(self._h, _ptr(k_new), _ptr(v_new), _ptr(k_pages), _ptr(v_pages),
                                            _ptr(block_table), int(prefix_len), _ptr(branch_lens), int(n_branches),
                                            int(rows)), "tts_kv_append")

    def tts_kv_rollback(self, branch_lens, accepted_len, n_branches: int, gamma: int):
        self._check(self._lib.tts_kv_rollback(self._h, _ptr(branch_lens), _ptr(accepted_len), int(n_branches),
                                              int(gamma)), "tts_kv_rollback")

    def tts_last_status(self) -> int:
        st = c_int(0)
        self._check(self._lib.tts_last_status(self._h, byref(st)), "tts_last_status")
        return st.value

    def tts_debug_wait_timeout(self, limit_ns: int):
        self._check(self._lib.tts_debug_wait_timeout(self._h, int(limit_ns)), "tts_debug_wait_timeout")

    def tts_profile_enable(self, on: bool):
        self._check(self._lib.tts_profile_enable(self._h, 1 if on else 0), "tts_profile_enable")

    def tts_profile_read(self):
        """(mean main-kernel us, mean merge-kernel us, calls recorded)."""
        a, b, n = c_float(0), c_float(0), c_int(0)
        self._check(self._lib.tts_profile_read(self._h, byref(a), byref(b), byref(n)), "tts_profile_read")
        return a.value, b.value, n.value

    def tts_launch_count(self) -> int:
        return int(self._lib.tts_launch_count(self._h))

    def tts_verify_step_host(self, n_layers: int, q_host, k_pools: Sequence, v_pools: Sequence, block_table_host,
                             prefix_len: int, branch_lens_host, n_branches: int, gamma: int, p_target_host,
                             q_draft_host, draft_tokens_host, uniforms_host, vocab: int, out_host,
                             accepted_len_host, next_token_host):
        ka = (c_void_p * n_layers)(*[_ptr(k).value for k in k_pools])
        va = (c_void_p * n_layers)(*[_ptr(v).value for v in v_pools])
        self._check(self._lib.tts_verify_step_host(
            self._h, int(n_layers), _ptr(q_host), ka, va, _ptr(block_table_host), int(prefix_len),
            _ptr(branch_lens_host), int(n_branches), int(gamma), _ptr(p_target_host), _ptr(q_draft_host),
            _ptr(draft_tokens_host), _ptr(uniforms_host), int(vocab), _ptr(out_host), _ptr(accepted_len_host),
            _ptr(next_token_host)), "tts_verify_step_host")


def _step_host_logits(self, n_layers: int, q_host, k_pools: Sequence, v_pools: Sequence, block_table_host,
                      prefix_len: int, branch_lens_host, n_branches: int, gamma: int, target_logits_host,
                      draft_logits_host, logits_dtype: int, draft_tokens_host, uniforms_host, vocab: int, out_host,
                      accepted_len_host, next_token_host):
    ka = (c_void_p * n_layers)(*[_ptr(k).value for k in k_pools])
    va = (c_void_p * n_layers)(*[_ptr(v).value for v in v_pools])
    self._check(self._lib.tts_verify_step_host_logits(
        self._h, int(n_layers), _ptr(q_host), ka, va, _ptr(block_table_host), int(prefix_len),
        _ptr(branch_lens_host), int(n_branches), int(gamma), _ptr(target_logits_host), _ptr(draft_logits_host),
        int(logits_dtype), _ptr(draft_tokens_host), _ptr(uniforms_host), int(vocab), _ptr(out_host),
        _ptr(accepted_len_host), _ptr(next_token_host)), "tts_verify_step_host_logits")


TtsContext.tts_verify_step_host_logits = _step_host_logits


def tts_verify_attn_noalloc(q, k_pages, v_pages, block_table, max_blocks_per_branch: int, prefix_len: int,
                            branch_lens, n_branches: int, gamma: int, n_q_heads: int, n_kv_heads: int, out,
                            stream=None):
    """Causal verify attention for callers that may not allocate device memory (no context, no
    cudaMalloc: the partial results live in a fixed array inside the library).  Raises TtsError with
    status -6 when the problem does not fit that array."""
    lib = load_library()
    handle = stream if isinstance(stream, int) or stream is None else stream.cuda_stream
    rc = lib.tts_verify_attn_noalloc(_ptr(q), _ptr(k_pages), _ptr(v_pages), _ptr(block_table),
                                     int(max_blocks_per_branch), int(prefix_len), _ptr(branch_lens),
                                     int(n_branches), int(gamma), int(n_q_heads), int(n_kv_heads), _ptr(out),
                                     c_void_p(handle or 0))
    if rc != 0:
        raise TtsError(rc, "tts_verify_attn_noalloc")


# -- host-only helpers (no context) -----------------------------------------------------------
def _vote(fn_name: str, answers, weights):
    lib = load_library()
    n = len(answers)
    a = (c_int64 * n)(*[int(x) for x in answers])
    w = (c_float * n)(*[float(x) for x in weights]) if weights is not None else None
    winner, votes = c_int64(0), c_int(0)
    rc = getattr(lib, fn_name)(a, w, n, byref(winner), byref(votes))
    if rc != 0:
        raise TtsError(rc, fn_name)
    return int(winner.value), int(votes.value)


def tts_majority_vote(answers, weights=None):
    """(winner, votes) over the branches' answers; optional weights give the weighted vote."""
    return _vote("tts_majority_vote", answers, weights)


def tts_confidence_max(answers, weights):
    """(answer of the most confident branch, branches that gave it)."""
    return _vote("tts_confidence_max", answers, weights)


def _limits(max_branches, max_gamma, max_steps):
    if max_branches is None and max_gamma is None and max_steps is None:
        return None
    return byref(TtsSearchLimits(64 if max_branches is None else int(max_branches),
                                 7 if max_gamma is None else int(max_gamma), int(max_steps or 0)))


def tts_greedy_search(tts_task, max_branches=None, max_gamma=None, max_steps=None):
    """Greedy (B, gamma) search over a Python callable tts_task(B, gamma) -> accuracy (negative =
    unavailable).  Returns (B, gamma, accuracy, steps, evaluations)."""
    lib = load_library()
    cb = _TASK_FN(lambda b, g, _u: float(tts_task(b, g)))
    B, G, acc, steps, evals = c_int(0), c_int(0), c_double(0.0), c_int(0), c_int(0)
    rc = lib.tts_greedy_search(cb, None, _limits(max_branches, max_gamma, max_steps), byref(B), byref(G), byref(acc),
                               byref(steps), byref(evals))
    if rc != 0:
        raise TtsError(rc, "tts_greedy_search")
    return B.value, G.value, acc.value, steps.value, evals.value


def tts_grid_search(tts_task, max_branches=None, max_gamma=None):
    """Exhaustive (B, gamma) search.  Returns (B, gamma, accuracy, evaluations)."""
    lib = load_library()
    cb = _TASK_FN(lambda b, g, _u: float(tts_task(b, g)))
    B, G, acc, evals = c_int(0), c_int(0), c_double(0.0), c_int(0)
    rc = lib.tts_grid_search(cb, None, _limits(max_branches, max_gamma, None), byref(B), byref(G), byref(acc),
                             byref(evals))
    if rc != 0:
        raise TtsError(rc, "tts_grid_search")
    return B.value, G.value, acc.value, evals.value
