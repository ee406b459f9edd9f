"""B200-native Pulsar Attention context encoding (selection, Phase 1, Phase 2).

The compute lives in a C-ABI CUDA library (``include/pulsar.h``); ``binding``
marshals device pointers into it.  Importing the package does not load the
library; the first use of a binding function does, and raises if it is missing.
"""
from . import cost_model, workloads  # noqa: F401

_BINDING_NAMES = (
    "pulsar_maxidf_select", "pulsar_phase1_attn", "pulsar_phase2_attn", "pulsar_lse_merge",
    "pulsar_phase2_generate_step", "pulsar_maxidf_select_noalloc",
    "maxidf_select_workspace_bytes", "phase1_workspace_bytes", "phase2_workspace_bytes",
    "PulsarError", "library_path", "load_library",
)


def __getattr__(name):
    if name == "binding" or name in _BINDING_NAMES:
        import importlib
        mod = importlib.import_module(".binding", __name__)
        return mod if name == "binding" else getattr(mod, name)
    raise AttributeError(name)
