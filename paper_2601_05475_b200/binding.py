"""ctypes binding of the C-ABI library (include/maxcode_attn.h, maxcode_search.h, maxcode_qkv.h): same names, argument marshalling only.

Device buffers are torch tensors (torch is used for device memory and streams only); every entry point
takes raw device pointers.  There is no fallback: if the shared library is missing or fails to load,
`lib()` raises.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, byref, c_char_p, c_double, c_float, c_int32, c_size_t, c_uint64, c_void_p

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libmaxcode_attn.so")
_lib = None

MC_OK, MC_ERR_INVALID_ARG, MC_ERR_UNSUPPORTED, MC_ERR_OUT_OF_MEMORY, MC_ERR_WORKSPACE_TOO_SMALL, MC_ERR_CUDA, \
    MC_ERR_TIMEOUT = range(7)
MC_F32, MC_BF16, MC_FP8_E4M3 = 0, 1, 2


class LayoutDesc(ctypes.Structure):
    _fields_ = [(n, c_int32) for n in ("num_groups", "batch", "num_q_heads", "num_kv_heads", "head_dim", "page_size",
                                       "num_pages", "max_prefix_pages", "max_suffix_pages", "dtype")] + \
               [(n, c_void_p) for n in ("k_pool", "v_pool", "group_offsets", "prefix_pages", "prefix_len",
                                        "suffix_pages", "suffix_len", "k_scale", "v_scale")]


class PrefixLevel(ctypes.Structure):
    _fields_ = [("num_groups", c_int32), ("max_pages", c_int32), ("group_offsets", c_void_p), ("pages", c_void_p),
                ("len", c_void_p), ("row_limit", c_void_p)]


class PartGeometry(ctypes.Structure):
    _fields_ = [(n, c_int32) for n in ("rows", "n_parts", "n_prefix_parts", "prefix_part_tokens",
                                       "suffix_part_tokens", "head_dim", "prefix_ctas")]


EXPORTS = {
    "mc_kv_layout_create": (c_int32, [POINTER(LayoutDesc), POINTER(c_void_p)]),
    "mc_kv_layout_create_cascade": (c_int32, [POINTER(LayoutDesc), POINTER(PrefixLevel), c_int32, POINTER(c_void_p)]),
    "mc_kv_layout_destroy": (c_int32, [c_void_p]),
    "mc_kv_layout_validate": (c_int32, [c_void_p, c_void_p, c_size_t, c_void_p]),
    "mc_kv_layout_refresh_prefix": (c_int32, [c_void_p, c_void_p]),
    "mc_kv_layout_refresh_tables": (c_int32, [c_void_p, c_void_p]),
    "mc_kv_layout_geometry": (c_int32, [c_void_p, POINTER(PartGeometry)]),
    "mc_workspace_bytes": (c_size_t, [c_void_p]),
    "mc_kv_append": (c_int32, [c_void_p, c_void_p, c_void_p, c_void_p]),
    "mc_kv_append_rope": (c_int32, [c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_double, c_void_p]),
    "mc_kv_append_tokens": (c_int32, [c_void_p, c_void_p, c_void_p, c_int32, c_void_p, c_void_p, c_void_p, c_double,
                                      c_void_p]),
    "mc_prefix_attn": (c_int32, [c_void_p, c_void_p, c_float, c_void_p, c_void_p, c_void_p]),
    "mc_suffix_attn": (c_int32, [c_void_p, c_void_p, c_float, c_void_p, c_void_p, c_void_p]),
    "mc_merge_lse": (c_int32, [c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]),
    "mc_decode_attn": (c_int32, [c_void_p, c_void_p, c_float, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]),
    "mc_decode_step": (c_int32, [c_void_p, c_void_p, c_void_p, c_void_p, c_float, c_void_p, c_void_p, c_void_p, c_size_t,
                                 c_void_p]),
    "mc_decode_step_host": (c_int32, [c_void_p, c_void_p, c_void_p, c_void_p, c_float, c_void_p, c_void_p,
                                      c_void_p, c_size_t, c_void_p]),
    "mc_decode_attn_static": (c_int32, [POINTER(LayoutDesc), c_void_p, c_float, c_void_p, c_void_p, c_void_p, c_void_p]),
    "mc_static_scratch_bytes": (c_size_t, []),
    "mc_get_last_status": (c_int32, [c_void_p, c_void_p]),
    "mc_hbm_read_probe": (c_int32, [c_void_p, c_size_t, c_void_p, c_void_p]),
    "mc_launch_count": (c_uint64, []),
    "mc_status_string": (c_char_p, [c_int32]),
    "mc_search_returns": (c_int32, [c_void_p, c_void_p, c_void_p, c_int32, c_int32, c_float, c_float, c_float, c_float,
                                    c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]),
    "mc_search_value_head": (c_int32, [c_void_p, c_int32, c_void_p, c_void_p, c_void_p]),
    "mc_search_group_argmax": (c_int32, [c_void_p, c_void_p, c_int32, c_void_p, c_void_p]),
    "mc_search_select": (c_int32, [c_void_p, c_void_p, c_void_p, c_int32, c_void_p, c_void_p, c_void_p, c_void_p,
                                   c_void_p]),
    "mc_qkv_plan_create": (c_int32, [c_void_p, c_void_p, c_void_p, c_int32, POINTER(c_void_p)]),
    "mc_qkv_plan_destroy": (c_int32, [c_void_p]),
    "mc_qkv_plan_geometry": (c_int32, [c_void_p, POINTER(c_int32), POINTER(c_int32), POINTER(c_size_t)]),
    "mc_qkv_append": (c_int32, [c_void_p, c_void_p, c_void_p, c_void_p, c_double, c_void_p]),
}


def lib_path() -> str:
    return _LIB_PATH


def lib() -> ctypes.CDLL:
    """The loaded shared library.  Raises if it has not been built (python -m paper_2601_05475_b200.build)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError("%s is missing: build it with `python -m paper_2601_05475_b200.build`; "
                               "there is no fallback path" % _LIB_PATH)
        l = ctypes.CDLL(_LIB_PATH)
        for name, (res, args) in EXPORTS.items():
            fn = getattr(l, name)
            fn.restype, fn.argtypes = res, args
        _lib = l
    return _lib


class McError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s: %s (status %d)" % (where, mc_status_string(status), status))


def _check(status: int, where: str) -> None:
    if status != MC_OK:
        raise McError(status, where)


def _ptr(x) -> int:
    """Raw address of a torch tensor (device or host), an int, or None."""
    if x is None:
        return 0
    if isinstance(x, int):
        return x
    return x.data_ptr()


def mc_status_string(status: int) -> str:
    return lib().mc_status_string(status).decode()


def mc_launch_count() -> int:
    return int(lib().mc_launch_count())


def mc_kv_layout_create(desc: LayoutDesc) -> int:
    h = c_void_p()
    _check(lib().mc_kv_layout_create(byref(desc), byref(h)), "mc_kv_layout_create")
    return h.value


def mc_kv_layout_create_cascade(desc: LayoutDesc, outer) -> int:
    """`outer`: sequence of PrefixLevel (outer cascade levels, any order)."""
    h = c_void_p()
    arr = (PrefixLevel * max(1, len(outer)))(*outer)
    _check(lib().mc_kv_layout_create_cascade(byref(desc), arr, len(outer), byref(h)), "mc_kv_layout_create_cascade")
    return h.value


def mc_kv_layout_destroy(layout: int) -> None:
    _check(lib().mc_kv_layout_destroy(layout), "mc_kv_layout_destroy")


def mc_kv_layout_refresh_prefix(layout: int, stream: int = 0) -> None:
    _check(lib().mc_kv_layout_refresh_prefix(layout, stream), "mc_kv_layout_refresh_prefix")


def mc_kv_layout_refresh_tables(layout: int, stream: int = 0) -> None:
    _check(lib().mc_kv_layout_refresh_tables(layout, stream), "mc_kv_layout_refresh_tables")


def mc_kv_layout_geometry(layout: int) -> PartGeometry:
    g = PartGeometry()
    _check(lib().mc_kv_layout_geometry(layout, byref(g)), "mc_kv_layout_geometry")
    return g


def mc_workspace_bytes(layout: int) -> int:
    return int(lib().mc_workspace_bytes(layout))


def mc_kv_layout_validate(layout: int, scratch, scratch_bytes: int, stream: int = 0) -> int:
    return lib().mc_kv_layout_validate(layout, _ptr(scratch), scratch_bytes, stream)


def mc_kv_append(layout: int, k_new, v_new, stream: int = 0) -> None:
    _check(lib().mc_kv_append(layout, _ptr(k_new), _ptr(v_new), stream), "mc_kv_append")


def mc_kv_append_rope(layout: int, k_new, v_new, q, pos_offset, theta_base: float, stream: int = 0) -> None:
    _check(lib().mc_kv_append_rope(layout, _ptr(k_new), _ptr(v_new), _ptr(q), _ptr(pos_offset), theta_base, stream),
           "mc_kv_append_rope")


def mc_kv_append_tokens(layout: int, k_new, v_new, n_max: int, n_new=None, q=None, pos_offset=None,
                        theta_base: float = 0.0, stream: int = 0) -> None:
    _check(lib().mc_kv_append_tokens(layout, _ptr(k_new), _ptr(v_new), n_max, _ptr(n_new), _ptr(q), _ptr(pos_offset),
                                     theta_base, stream), "mc_kv_append_tokens")


def mc_prefix_attn(layout: int, q, scale: float, o_part, lse_part, stream: int = 0) -> None:
    _check(lib().mc_prefix_attn(layout, _ptr(q), scale, _ptr(o_part), _ptr(lse_part), stream), "mc_prefix_attn")


def mc_suffix_attn(layout: int, q, scale: float, o_part, lse_part, stream: int = 0) -> None:
    _check(lib().mc_suffix_attn(layout, _ptr(q), scale, _ptr(o_part), _ptr(lse_part), stream), "mc_suffix_attn")


def mc_merge_lse(layout: int, o_part, lse_part, o, lse, stream: int = 0) -> None:
    _check(lib().mc_merge_lse(layout, _ptr(o_part), _ptr(lse_part), _ptr(o), _ptr(lse), stream), "mc_merge_lse")


def mc_decode_attn(layout: int, q, scale: float, o, lse, ws, ws_bytes: int, stream: int = 0) -> None:
    _check(lib().mc_decode_attn(layout, _ptr(q), scale, _ptr(o), _ptr(lse), _ptr(ws), ws_bytes, stream),
           "mc_decode_attn")


def mc_decode_step(layout: int, k_new, v_new, q, scale: float, o, lse, ws, ws_bytes: int, stream: int = 0) -> None:
    _check(lib().mc_decode_step(layout, _ptr(k_new), _ptr(v_new), _ptr(q), scale, _ptr(o), _ptr(lse), _ptr(ws),
                                ws_bytes, stream), "mc_decode_step")


def mc_decode_step_host(layout: int, k_new_host, v_new_host, q_host, scale: float, o_host, lse_host, ws,
                        ws_bytes: int, stream: int = 0) -> None:
    _check(lib().mc_decode_step_host(layout, _ptr(k_new_host), _ptr(v_new_host), _ptr(q_host), scale,
                                     _ptr(o_host), _ptr(lse_host), _ptr(ws), ws_bytes, stream),
           "mc_decode_step_host")


def mc_decode_attn_static(desc: LayoutDesc, q, scale: float, o, lse, dev_status=None, stream: int = 0) -> int:
    """The step without handle, workspace or allocation (scratch compiled into the library).  Returns the
    status code instead of raising, so callers can test for MC_ERR_WORKSPACE_TOO_SMALL."""
    return lib().mc_decode_attn_static(byref(desc), _ptr(q), scale, _ptr(o), _ptr(lse), _ptr(dev_status), stream)


def mc_static_scratch_bytes() -> int:
    return int(lib().mc_static_scratch_bytes())


def mc_hbm_read_probe(buf, nbytes: int, sink, stream: int = 0) -> None:
    _check(lib().mc_hbm_read_probe(_ptr(buf), nbytes, _ptr(sink), stream), "mc_hbm_read_probe")


def mc_get_last_status(layout: int, stream: int = 0) -> int:
    return lib().mc_get_last_status(layout, stream)


def mc_search_returns(speedup_pct, correct, length, N: int, T: int, s1: float, s2: float, s3: float, gamma: float,
                      reward=None, best_so_far=None, value_target=None, label=None, traj_return=None,
                      stream: int = 0) -> None:
    _check(lib().mc_search_returns(_ptr(speedup_pct), _ptr(correct), _ptr(length), N, T, s1, s2, s3, gamma, _ptr(reward),
                                   _ptr(best_so_far), _ptr(value_target), _ptr(label), _ptr(traj_return), stream),
           "mc_search_returns")


def mc_search_value_head(logits, N: int, prob, expected, stream: int = 0) -> None:
    _check(lib().mc_search_value_head(_ptr(logits), N, _ptr(prob), _ptr(expected), stream), "mc_search_value_head")


def mc_search_group_argmax(values, group_offsets, P: int, best, stream: int = 0) -> None:
    _check(lib().mc_search_group_argmax(_ptr(values), _ptr(group_offsets), P, _ptr(best), stream),
           "mc_search_group_argmax")


def mc_search_select(logits, traj_return, group_offsets, P: int, prob=None, expected=None, best_return=None,
                     best_expected=None, stream: int = 0) -> None:
    _check(lib().mc_search_select(_ptr(logits), _ptr(traj_return), _ptr(group_offsets), P, _ptr(prob), _ptr(expected),
                                  _ptr(best_return), _ptr(best_expected), stream), "mc_search_select")


def mc_qkv_plan_create(layout: int, w_qkv, bias, hidden: int) -> int:
    h = c_void_p()
    _check(lib().mc_qkv_plan_create(layout, _ptr(w_qkv), _ptr(bias), hidden, byref(h)), "mc_qkv_plan_create")
    return h.value


def mc_qkv_plan_destroy(plan: int) -> None:
    _check(lib().mc_qkv_plan_destroy(plan), "mc_qkv_plan_destroy")


def mc_qkv_plan_geometry(plan: int):
    """(splits, ctas, workspace_bytes)"""
    s, c, w = c_int32(), c_int32(), c_size_t()
    _check(lib().mc_qkv_plan_geometry(plan, byref(s), byref(c), byref(w)), "mc_qkv_plan_geometry")
    return s.value, c.value, w.value


def mc_qkv_append(plan: int, x, q_out, pos_offset=None, theta_base: float = 0.0, stream: int = 0) -> None:
    _check(lib().mc_qkv_append(plan, _ptr(x), _ptr(q_out), _ptr(pos_offset), theta_base, stream), "mc_qkv_append")
