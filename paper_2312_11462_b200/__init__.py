"""Review-step hot path of Cascade Speculative Drafting (arXiv 2312.11462) for sm_100a.

`paper_2312_11462_b200.binding` is the ctypes binding of the C ABI (include/csd.h); it loads
`libcsd.so`, which `paper_2312_11462_b200.build` compiles with nvcc.  Attribute access on the
package forwards to the binding and raises if the library has not been built: there is no
fallback path.
"""
__all__ = ["binding", "build"]


def __getattr__(name):
    if name in ("binding", "build"):
        import importlib
        return importlib.import_module(f"{__name__}.{name}")
    from . import binding
    return getattr(binding, name)
