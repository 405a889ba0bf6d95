"""B200-native adapted quantized linear layer (Q-BLoRA / QA-BLoRA, arXiv 2407.17029).

``paper_2407_17029_b200.synth``   seeded synthetic inputs (numpy only)
``paper_2407_17029_b200.binding`` ctypes binding of the C-ABI CUDA library (loaded lazily)
"""
import importlib

__all__ = ["synth", "binding"]


def __getattr__(name):
    if name in __all__:
        return importlib.import_module(f"{__name__}.{name}")
    raise AttributeError(name)
