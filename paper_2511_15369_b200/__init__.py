"""B200-native integer-only non-linear layers of IPTQ-ViT (Softmax / GELU / LayerNorm
and the fused INT8 attention / MLP blocks), exposed through a C-ABI CUDA library.

``paper_2511_15369_b200.api`` is the thin Python binding (argument marshalling only);
``paper_2511_15369_b200.synth`` draws the seeded synthetic workloads.  The binding is
imported lazily so that the workload generator can be used without the CUDA library.
"""
__all__ = ["api", "synth"]


def __getattr__(name):
    if name in ("api", "synth"):
        import importlib
        return importlib.import_module("." + name, __name__)
    raise AttributeError(name)
