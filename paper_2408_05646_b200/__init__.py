"""B200-native Eigen Attention: rank-r KV cache, split-KV decode and causal prefill.

The compute lives in `libeigenattn.so` (hand-written sm_100a CUDA behind a C ABI,
declared in include/eigen_attn.h).  `binding` marshals arguments to it; `synth`
draws seeded synthetic inputs.  There is no CPU fallback: using the binding
without the built library raises.
"""

__all__ = ["binding", "synth"]


def __getattr__(name):
    if name in __all__:
        import importlib
        return importlib.import_module(f"{__name__}.{name}")
    raise AttributeError(name)
