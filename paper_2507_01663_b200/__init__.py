"""B200-native GRPO scoring path (pack -> fused LM-head log-prob -> advantage -> policy loss).

``workloads`` (synthetic inputs) imports without the CUDA library; everything else loads
``libasyncflow.so`` on first use and raises if it is missing -- there is no CPU fallback.
"""

__all__ = ["Context", "AfError", "load_library", "new_loss_out", "read_loss_out", "workloads"]


def __getattr__(name):
    if name in ("Context", "AfError", "load_library", "new_loss_out", "read_loss_out", "binding"):
        import importlib
        binding = importlib.import_module(".binding", __name__)
        return binding if name == "binding" else getattr(binding, name)
    if name == "workloads":
        import importlib
        return importlib.import_module(".workloads", __name__)
    raise AttributeError(name)
