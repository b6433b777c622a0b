"""ctypes binding of the C ABI in include/vvs.h: same function names, argument marshalling only.

Tensors are torch CUDA tensors used purely as device memory (`data_ptr()`); every step of the
verification runs in the library's CUDA kernels.  There is no CPU fallback: if the shared
library has not been built, importing this module raises.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "lib", "libvvs.so")
if not os.path.exists(_LIB_PATH):
    raise ImportError(
        f"{_LIB_PATH} is missing: build it first (python -m paper_2511_13587_b200.build, or "
        "__graft_entry__.build()).  There is no fallback path.")
lib = C.CDLL(_LIB_PATH)

VVS_OK = 0
VVS_DTYPE_FP32, VVS_DTYPE_BF16 = 0, 1
VVS_ROPE_NONE, VVS_ROPE_1D, VVS_ROPE_2D_GRID = 0, 1, 2
VVS_MODE_STRICT, VVS_MODE_RELAXED = 0, 1
VVS_DEV_BAD_TOKEN, VVS_DEV_CACHE_OVERFLOW, VVS_DEV_BAD_NEIGHBOUR = 1, 2, 4
VVS_DEV_TIMEOUT, VVS_DEV_FCACHE_MISS, VVS_DEV_BAD_ARG = 8, 16, 32


class vvs_model_desc(C.Structure):
    _fields_ = [(n, C.c_int32) for n in (
        "n_layers", "d_model", "n_heads", "head_dim", "d_ff", "vocab", "vocab_offset", "lm_rows",
        "tok_rows", "s_max", "rope_mode", "rope_grid_w", "n_prefix", "dtype", "max_rows",
        "max_block", "max_nbr_k")] + [("rms_eps", C.c_float), ("rope_base", C.c_float),
                                      ("deterministic", C.c_int32)]


class vvs_layer_weights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("w_qkv", "w_o", "w_gate", "w_up", "w_down", "norm1", "norm2")]


class vvs_weights(C.Structure):
    _fields_ = [("tok_emb", C.c_void_p), ("norm_f", C.c_void_p), ("w_lm", C.c_void_p),
                ("layers", C.POINTER(vvs_layer_weights))]


class vvs_verify_args(C.Structure):
    _fields_ = [("n_images", C.c_int32), ("n_cfg", C.c_int32), ("n_forced", C.c_int32),
                ("n_draft_max", C.c_int32), ("block", C.c_void_p), ("n_draft", C.c_void_p),
                ("kv_k", C.c_void_p), ("kv_v", C.c_void_p), ("kv_rows", C.c_int32),
                ("cache_len", C.c_void_p), ("cache_len_host", C.c_void_p),
                ("draft_probs", C.c_void_p), ("uniforms", C.c_void_p), ("cfg_scale", C.c_float),
                ("temperature", C.c_float), ("mode", C.c_int32), ("nbr_k", C.c_int32),
                ("delta", C.c_float), ("tree_parent", C.c_void_p), ("adjusted_residual", C.c_int32)]


class vvs_verify_out(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("accept_len", "next_token", "new_len", "n_commit", "accept_mask",
                                          "target_probs", "hidden", "accept_path",
                                          "margins")]


class vvs_fcache(C.Structure):
    _fields_ = [("feat", C.c_void_p), ("fpos", C.c_void_p), ("newest", C.c_void_p),
                ("n_rows", C.c_int32), ("cap", C.c_int32)]


_P = C.c_void_p
lib.vvs_create.argtypes = [C.POINTER(vvs_model_desc), C.POINTER(_P)]
lib.vvs_destroy.argtypes = [_P]
lib.vvs_workspace_bytes.argtypes = [C.POINTER(vvs_model_desc), C.POINTER(C.c_size_t)]
lib.vvs_bind_weights.argtypes = [_P, C.POINTER(vvs_weights)]
lib.vvs_bind_neighbors.argtypes = [_P, _P, _P, C.c_int64]
lib.vvs_verify.argtypes = [_P, C.POINTER(vvs_verify_args), C.POINTER(vvs_verify_out), _P]
lib.vvs_epilogue.argtypes = [_P, _P, C.c_int32, C.c_int32, _P, C.POINTER(vvs_verify_args),
                             C.POINTER(vvs_verify_out), _P]
lib.vvs_decide.argtypes = [_P, _P, C.c_int32, C.c_int32, _P, C.POINTER(vvs_verify_args),
                           C.POINTER(vvs_verify_out), _P]
lib.vvs_decide.restype = C.c_int
lib.vvs_decide_noalloc.argtypes = [_P, C.c_int32, C.c_int32, C.c_int32, C.c_int32, _P, _P, _P,
                                   C.POINTER(vvs_verify_args), C.POINTER(vvs_verify_out), _P, _P]
lib.vvs_decide_noalloc.restype = C.c_int
lib.vvs_selftest_bounded_wait.argtypes = [_P, _P, C.POINTER(C.c_int32)]
lib.vvs_feature_cache_reset.argtypes = [_P, C.POINTER(vvs_fcache), _P]
lib.vvs_feature_cache_store.argtypes = [_P, C.POINTER(vvs_fcache), _P, C.c_int32, _P, _P, _P]
lib.vvs_feature_cache_fetch.argtypes = [_P, C.POINTER(vvs_fcache), _P, C.c_int32, _P, C.c_int32,
                                        C.c_int32, _P, _P, _P]
lib.vvs_skip_decide.argtypes = [_P, _P, _P, C.c_int32, C.c_int32, C.c_int32, _P, C.c_int32, C.c_int32, _P,
                                C.c_int32, C.c_float, C.c_float, _P, _P, _P]
lib.vvs_skip_decide.restype = C.c_int
lib.vvs_select_unverified.argtypes = [_P, _P, _P, C.c_int32, C.c_int32, C.c_int32, _P, _P, _P, _P, _P]
lib.vvs_select_unverified.restype = C.c_int
lib.vvs_device_status.argtypes = [_P, _P, C.POINTER(C.c_int32)]
lib.vvs_last_launch_count.argtypes = [_P]
lib.vvs_profile_enable.argtypes = [_P, C.c_int]
lib.vvs_profile_read.argtypes = [_P, _P, C.POINTER(C.c_float), C.POINTER(C.c_int32)]
lib.vvs_strerror.argtypes = [C.c_int]
lib.vvs_strerror.restype = C.c_char_p
for _n in ("vvs_create", "vvs_destroy", "vvs_workspace_bytes", "vvs_bind_weights",
           "vvs_bind_neighbors", "vvs_verify", "vvs_epilogue", "vvs_feature_cache_reset",
           "vvs_feature_cache_store", "vvs_feature_cache_fetch", "vvs_device_status",
           "vvs_last_launch_count", "vvs_profile_enable", "vvs_profile_read"):
    getattr(lib, _n).restype = C.c_int


class VvsError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {vvs_strerror(status)} ({status})")


def vvs_strerror(status: int) -> str:
    return lib.vvs_strerror(int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != VVS_OK:
        raise VvsError(status, where)


def _ptr(t):
    """Device (or host) address of a tensor, None -> NULL."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream):
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def make_desc(shape, max_rows: int, max_block: int, max_nbr_k: int = 1,
              deterministic: bool = True) -> vvs_model_desc:
    """Fill a vvs_model_desc from any object with the ModelShape attribute names."""
    d = vvs_model_desc()
    for name in ("n_layers", "d_model", "n_heads", "head_dim", "d_ff", "vocab", "vocab_offset",
                 "lm_rows", "tok_rows", "s_max", "rope_mode", "rope_grid_w", "n_prefix", "dtype"):
        setattr(d, name, int(getattr(shape, name)))
    d.rms_eps = float(shape.rms_eps)
    d.rope_base = float(shape.rope_base)
    d.max_rows, d.max_block, d.max_nbr_k = int(max_rows), int(max_block), int(max_nbr_k)
    d.deterministic = 1 if deterministic else 0
    return d


_keepalive: dict[int, dict] = {}


def vvs_workspace_bytes(desc: vvs_model_desc) -> int:
    out = C.c_size_t(0)
    _check(lib.vvs_workspace_bytes(C.byref(desc), C.byref(out)), "vvs_workspace_bytes")
    return out.value


def vvs_create(desc: vvs_model_desc) -> int:
    ctx = _P()
    _check(lib.vvs_create(C.byref(desc), C.byref(ctx)), "vvs_create")
    _keepalive[ctx.value] = {}
    return ctx.value


def vvs_destroy(ctx: int) -> None:
    _keepalive.pop(ctx, None)
    _check(lib.vvs_destroy(ctx), "vvs_destroy")


def vvs_bind_weights(ctx: int, weights: dict) -> None:
    """weights: {'tok_emb', 'norm_f', 'w_lm': tensor, 'layers': [ {w_qkv, w_o, w_gate, w_up,
    w_down, norm1, norm2: tensor}, ... ]} of CUDA tensors (kept alive until vvs_destroy)."""
    layers = weights.get("layers") or []
    arr = (vvs_layer_weights * max(1, len(layers)))()
    for i, lw in enumerate(layers):
        for n, _ in vvs_layer_weights._fields_:
            setattr(arr[i], n, _ptr(lw[n]))
    w = vvs_weights(_ptr(weights.get("tok_emb")), _ptr(weights.get("norm_f")), _ptr(weights["w_lm"]),
                    C.cast(arr, C.POINTER(vvs_layer_weights)))
    _check(lib.vvs_bind_weights(ctx, C.byref(w)), "vvs_bind_weights")
    _keepalive[ctx]["weights"] = weights


def vvs_bind_neighbors(ctx: int, row_ptr: torch.Tensor, col: torch.Tensor) -> None:
    _check(lib.vvs_bind_neighbors(ctx, _ptr(row_ptr), _ptr(col), int(col.numel())), "vvs_bind_neighbors")
    _keepalive[ctx]["nbr"] = (row_ptr, col)


def _args(n_images, n_cfg, n_forced, n_draft_max, block, n_draft, kv_k, kv_v, kv_rows, cache_len,
          cache_len_host, draft_probs, uniforms, cfg_scale, temperature, mode, nbr_k, delta,
          tree_parent=None, adjusted_residual=False):
    return vvs_verify_args(int(n_images), int(n_cfg), int(n_forced), int(n_draft_max), _ptr(block),
                           _ptr(n_draft), _ptr(kv_k), _ptr(kv_v), int(kv_rows), _ptr(cache_len),
                           _ptr(cache_len_host), _ptr(draft_probs), _ptr(uniforms), float(cfg_scale),
                           float(temperature), int(mode), int(nbr_k), float(delta), _ptr(tree_parent),
                           int(adjusted_residual))


def _out(accept_len, next_token, new_len, n_commit, accept_mask, target_probs, hidden, margins,
         accept_path=None):
    return vvs_verify_out(_ptr(accept_len), _ptr(next_token), _ptr(new_len), _ptr(n_commit), _ptr(accept_mask),
                          _ptr(target_probs), _ptr(hidden), _ptr(accept_path), _ptr(margins))


def vvs_verify(ctx: int, *, n_images, n_cfg, n_forced, n_draft_max, block, kv_k, kv_v, kv_rows,
               cache_len, draft_probs, uniforms, accept_len, next_token, new_len, n_draft=None,
               cache_len_host=None, cfg_scale=1.0, temperature=1.0, mode=VVS_MODE_STRICT, nbr_k=1,
               delta=float("inf"), n_commit=None, accept_mask=None, target_probs=None, hidden=None,
               margins=None, tree_parent=None, accept_path=None, adjusted_residual=False, stream=None) -> None:
    a = _args(n_images, n_cfg, n_forced, n_draft_max, block, n_draft, kv_k, kv_v, kv_rows, cache_len,
              cache_len_host, draft_probs, uniforms, cfg_scale, temperature, mode, nbr_k, delta, tree_parent,
              adjusted_residual)
    o = _out(accept_len, next_token, new_len, n_commit, accept_mask, target_probs, hidden, margins, accept_path)
    _check(lib.vvs_verify(ctx, C.byref(a), C.byref(o), _stream(stream)), "vvs_verify")


def vvs_epilogue(ctx: int, *, hidden_in, n_rows_per_seq, first_row, drafts, n_images, n_cfg,
                 n_draft_max, draft_probs, uniforms, accept_len, next_token, n_draft=None,
                 cfg_scale=1.0, temperature=1.0, mode=VVS_MODE_STRICT, nbr_k=1, delta=float("inf"),
                 accept_mask=None, target_probs=None, margins=None, adjusted_residual=False,
                 stream=None) -> None:
    a = _args(n_images, n_cfg, 1, n_draft_max, None, n_draft, None, None, 0, None, None, draft_probs,
              uniforms, cfg_scale, temperature, mode, nbr_k, delta, None, adjusted_residual)
    o = _out(accept_len, next_token, None, None, accept_mask, target_probs, None, margins)
    _check(lib.vvs_epilogue(ctx, _ptr(hidden_in), int(n_rows_per_seq), int(first_row), _ptr(drafts),
                            C.byref(a), C.byref(o), _stream(stream)), "vvs_epilogue")


def vvs_decide(ctx: int, *, target_probs, n_rows_per_seq, first_row, drafts, n_images, n_draft_max,
               draft_probs, uniforms, accept_len, next_token, n_draft=None, mode=VVS_MODE_STRICT,
               nbr_k=1, delta=float("inf"), accept_mask=None, margins=None, tree_parent=None,
               accept_path=None, adjusted_residual=False, stream=None) -> None:
    a = _args(n_images, 1, 1, n_draft_max, None, n_draft, None, None, 0, None, None, draft_probs,
              uniforms, 1.0, 1.0, mode, nbr_k, delta, tree_parent, adjusted_residual)
    o = _out(accept_len, next_token, None, None, accept_mask, None, None, margins, accept_path)
    _check(lib.vvs_decide(ctx, _ptr(target_probs), int(n_rows_per_seq), int(first_row), _ptr(drafts),
                          C.byref(a), C.byref(o), _stream(stream)), "vvs_decide")


def vvs_decide_noalloc(*, target_probs, vocab, vocab_offset, n_rows_per_seq, first_row, drafts,
                       n_images, n_draft_max, draft_probs, uniforms, accept_len, next_token,
                       nbr_row_ptr=None, nbr_col=None, n_draft=None, mode=VVS_MODE_STRICT, nbr_k=1,
                       delta=float("inf"), accept_mask=None, margins=None, status_bits=None,
                       tree_parent=None, accept_path=None, adjusted_residual=False, stream=None) -> None:
    """vvs_decide for callers that must not allocate device memory: no context, scratch in a fixed
    device array inside the library (limits: 64 images, 16 drafts, 64 neighbours, vocab 65536;
    chains only: tree_parent / accept_path are refused).  Calls on one device share that array
    and must not overlap on the GPU."""
    a = _args(n_images, 1, 1, n_draft_max, None, n_draft, None, None, 0, None, None, draft_probs,
              uniforms, 1.0, 1.0, mode, nbr_k, delta, tree_parent, adjusted_residual)
    o = _out(accept_len, next_token, None, None, accept_mask, None, None, margins, accept_path)
    _check(lib.vvs_decide_noalloc(_ptr(target_probs), int(vocab), int(vocab_offset), int(n_rows_per_seq),
                                  int(first_row), _ptr(drafts), _ptr(nbr_row_ptr), _ptr(nbr_col),
                                  C.byref(a), C.byref(o), _ptr(status_bits), _stream(stream)),
           "vvs_decide_noalloc")


def vvs_selftest_bounded_wait(ctx: int, stream=None):
    """Runs the bounded-wait self-test kernel; returns the two give-up flags."""
    out = (C.c_int32 * 2)()
    _check(lib.vvs_selftest_bounded_wait(ctx, _stream(stream), out), "vvs_selftest_bounded_wait")
    return int(out[0]), int(out[1])


def make_fcache(feat: torch.Tensor, fpos: torch.Tensor, newest: torch.Tensor) -> vvs_fcache:
    """feat [n_rows, cap, d], fpos int32 [n_rows, cap], newest int32 [n_rows] (CUDA tensors)."""
    fc = vvs_fcache(_ptr(feat), _ptr(fpos), _ptr(newest), int(feat.shape[0]), int(feat.shape[1]))
    fc._keep = (feat, fpos, newest)
    return fc


def vvs_feature_cache_reset(ctx: int, fc: vvs_fcache, stream=None) -> None:
    _check(lib.vvs_feature_cache_reset(ctx, C.byref(fc), _stream(stream)), "vvs_feature_cache_reset")


def vvs_feature_cache_store(ctx: int, fc: vvs_fcache, hidden, n_rows_per_seq, base_pos, n_store,
                            stream=None) -> None:
    _check(lib.vvs_feature_cache_store(ctx, C.byref(fc), _ptr(hidden), int(n_rows_per_seq),
                                       _ptr(base_pos), _ptr(n_store), _stream(stream)),
           "vvs_feature_cache_store")


def vvs_feature_cache_fetch(ctx: int, fc: vvs_fcache, skip_mask, n_images, gamma, gamma_max,
                            staleness, out, out_pos, stream=None) -> None:
    _check(lib.vvs_feature_cache_fetch(ctx, C.byref(fc), _ptr(skip_mask), int(n_images), _ptr(gamma),
                                       int(gamma_max), int(staleness), _ptr(out), _ptr(out_pos),
                                       _stream(stream)), "vvs_feature_cache_fetch")


def vvs_skip_decide(ctx: int, paths, path_len, codebook, last_verified, stride: int, alpha: float,
                    threshold: float, decision, similarity, stream=None) -> None:
    """Alg. 1 / Eq. 2 of the paper: paths int32 [B, N, L], path_len int32 [B, N] or None,
    codebook float32 [V, dim], last_verified uint8 [B] or None -> decision uint8 [B], similarity
    float32 [B]."""
    b, n, l = paths.shape
    v, dim = codebook.shape
    _check(lib.vvs_skip_decide(ctx, _ptr(paths), _ptr(path_len), int(b), int(n), int(l), _ptr(codebook), int(v),
                               int(dim), _ptr(last_verified), int(stride), float(alpha), float(threshold),
                               _ptr(decision), _ptr(similarity), _stream(stream)), "vvs_skip_decide")


def vvs_select_unverified(ctx: int, paths, path_len, uniforms, out_path, out_gamma, out_tokens, stream=None) -> None:
    """Sec. 4.2 / Eq. 3: uniform draw of one candidate path per image, cut to gamma tokens."""
    b, n, l = paths.shape
    _check(lib.vvs_select_unverified(ctx, _ptr(paths), _ptr(path_len), int(b), int(n), int(l), _ptr(uniforms),
                                     _ptr(out_path), _ptr(out_gamma), _ptr(out_tokens), _stream(stream)),
           "vvs_select_unverified")


def vvs_device_status(ctx: int, stream=None, raise_on_error: bool = False) -> int:
    bits = C.c_int32(0)
    rc = lib.vvs_device_status(ctx, _stream(stream), C.byref(bits))
    if raise_on_error:
        _check(rc, "vvs_device_status")
    return bits.value


def vvs_last_launch_count(ctx: int) -> int:
    return lib.vvs_last_launch_count(ctx)


def vvs_profile_enable(ctx: int, on: bool) -> None:
    _check(lib.vvs_profile_enable(ctx, 1 if on else 0), "vvs_profile_enable")


def vvs_profile_read(ctx: int, stream=None):
    """Returns ([ms per class], [launches per class]) accumulated since the last read;
    classes: 0 GEMM, 1 attention, 2 other, 3 whole-chain kernel."""
    ms = (C.c_float * 4)(0, 0, 0, 0)
    n = (C.c_int32 * 4)(0, 0, 0, 0)
    _check(lib.vvs_profile_read(ctx, _stream(stream), ms, n), "vvs_profile_read")
    return list(ms), list(n)
