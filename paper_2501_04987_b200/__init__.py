"""TreeKV (arXiv 2501.04987) hot path for NVIDIA B200: a C-ABI CUDA library and its thin Python binding.

`paper_2501_04987_b200.binding` loads libtreekv.so (built in-tree by `paper_2501_04987_b200._build`) and
exposes the functions of include/treekv.h under the same names, plus the `TreeKV` convenience class.
There is no CPU fallback: using the binding without the built library raises ImportError.
"""

__all__ = ["binding", "TreeKV"]


def __getattr__(name):
    if name == "binding":
        import importlib

        return importlib.import_module(".binding", __name__)
    if name == "TreeKV":
        from .binding import TreeKV

        return TreeKV
    raise AttributeError(name)
