"""AMS-KV hot path for NVIDIA B200: segmented per-layer KV cache, scale-adaptive attention
and inter-scale key similarity, as CUDA kernels behind a small C ABI (include/amskv.h).

`binding` mirrors the C ABI one to one; `synth` makes seeded synthetic workloads and needs
nothing but torch.  `binding` loads libamskv.so the first time it is touched (as
`paper_2511_16047_b200.binding`, or through any of its names on the package) and raises
ImportError if the library has not been built; `synth` can be imported without it.
"""
import importlib

from . import synth  # noqa: F401


def __getattr__(name):
    # binding (and the names it exports) on first use, so that importing the input generators
    # alone does not map the CUDA library
    binding = importlib.import_module(__name__ + ".binding")
    if name == "binding":
        return binding
    try:
        return getattr(binding, name)
    except AttributeError:
        raise AttributeError("module %r has no attribute %r" % (__name__, name)) from None
