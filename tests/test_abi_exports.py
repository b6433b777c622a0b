"""The C-ABI library builds for sm_100a without a GPU, loads, and exports every function that
include/vvs.h declares.  No compute call is made."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "vvs.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(vvs_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    from paper_2511_13587_b200 import build
    lib_path = build.build()
    lib = ctypes.CDLL(lib_path)
    names = _declared()
    assert {"vvs_verify", "vvs_epilogue", "vvs_feature_cache_store", "vvs_feature_cache_fetch",
            "vvs_create", "vvs_bind_weights", "vvs_bind_neighbors"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n
    lib.vvs_strerror.restype = ctypes.c_char_p
    assert lib.vvs_strerror(0) == b"ok"
    assert b"capacity" in lib.vvs_strerror(-4).lower()


def test_binding_structs_match_header_field_order():
    from paper_2511_13587_b200 import binding as vb
    text = open(os.path.join(ROOT, "include", "vvs.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    for struct in (vb.vvs_model_desc, vb.vvs_layer_weights, vb.vvs_weights, vb.vvs_verify_args,
                   vb.vvs_verify_out, vb.vvs_fcache):
        body = re.search(r"typedef struct %s \{(.*?)\}" % struct.__name__, text, flags=re.S).group(1)
        fields = re.findall(r"(\w+)\s*;", body)
        assert fields == [f[0] for f in struct._fields_], struct.__name__


def test_host_side_argument_errors_need_no_gpu():
    from paper_2511_13587_b200 import binding as vb
    from vvs_synth.configs import TINY
    d = vb.make_desc(TINY, 1, 5)
    assert vb.vvs_workspace_bytes(d) > 0
    d.max_block = 33
    out = ctypes.c_size_t(0)
    assert vb.lib.vvs_workspace_bytes(ctypes.byref(d), ctypes.byref(out)) == -2
    d = vb.make_desc(TINY, 1, 5)
    d.n_heads = 3
    assert vb.lib.vvs_workspace_bytes(ctypes.byref(d), ctypes.byref(out)) == -2
    d = vb.make_desc(TINY, 1, 5)
    d.vocab = 65535 * 128 + 1                   # beyond the LM head's grid
    d.lm_rows = d.vocab_offset + d.vocab
    assert vb.lib.vvs_workspace_bytes(ctypes.byref(d), ctypes.byref(out)) == -2
    assert vb.lib.vvs_workspace_bytes(None, ctypes.byref(out)) == -1
    assert vb.lib.vvs_verify(None, None, None, None) == -1
    assert vb.lib.vvs_destroy(None) == -1
