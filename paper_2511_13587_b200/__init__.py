"""B200 (sm_100a) verify step of VVS speculative decoding: CUDA kernels behind a C ABI
(include/vvs.h) plus a ctypes binding with the same function names.

`binding` is imported lazily so that `paper_2511_13587_b200.build` can be used before the
shared library exists.  There is no CPU fallback."""


def __getattr__(name):
    if name == "binding":
        import importlib
        return importlib.import_module(".binding", __name__)
    raise AttributeError(name)
