"""EF21 hot path on one B200: Python binding of the libef21 C ABI (see include/ef21.h).

The compiled library is loaded on first use of the binding; ``build.build()`` compiles it.
"""
__all__ = ["binding", "build"]


def __getattr__(name):
    if name in ("EF21", "topk", "Ef21Error", "workspace_bytes", "status_string",
                "INIT_COMPRESSED", "INIT_ZERO", "INIT_GRADIENT",
                "PATH_AUTO", "PATH_LAUNCHES", "PATH_PERSISTENT"):
        from . import binding
        return getattr(binding, name)
    raise AttributeError(name)
