"""Cleave hot path on one B200: plan -> grouped sub-GEMM execution -> assembly -> reissue.

Thin ctypes binding over the C-ABI library `lib/libcleave.so` (CUDA kernels for sm_100a).  The
binding only marshals arguments; every step runs in the library.  There is no fallback: the first
use of anything but the `build` submodule loads the library and raises if it has not been built.
"""
_BINDING_NAMES = ("CleaveError", "Plan", "default_opts", "lib", "lib_path", "plan", "plan_uniform",
                  "GEMM_DTYPE", "TASK_DTYPE", "DEVICE_DTYPE", "strerror", "EXEC_DIRECT", "EXEC_FINISH", "EXEC_BF16", "EXEC_CONSUME")


def __getattr__(name):
    # the binding is loaded on first use, so that `paper_2512_22142_b200.build` can be imported (and
    # run) before the library exists
    if name in _BINDING_NAMES or name == "binding":
        import importlib
        binding = importlib.import_module(".binding", __name__)
        return binding if name == "binding" else getattr(binding, name)
    raise AttributeError(f"module {__name__!r} has no attribute {name!r}")
