"""Lognormal neural-gradient compression for NVIDIA B200 (sm_100a).

The CUDA library is loaded on first use of any compute entry point
(``paper_2006_08173_b200.binding``); there is no CPU fallback.
"""

__all__ = ["binding", "synth"]


def __getattr__(name):
    if name == "binding":
        import importlib
        return importlib.import_module(__name__ + ".binding")
    raise AttributeError(name)
