"""B200-native (sm_100a) implementation of the LAGA per-rank attention hot path.

One sequence-parallel rank's compute after the latent all-gather (Algorithm 1 steps 4-5 of the
paper, and the backward of Section 5.2): head-shard up-projection of the gathered MLA latent,
key assembly with the shared rope band, explicit causal softmax attention, forward and backward.

The work is done by hand-written CUDA kernels behind a C ABI (``include/laga.h``); ``laga`` is the
ctypes binding (argument marshalling only).  The shared library is loaded on first use and its
absence is an error: there is no CPU or eager fallback.
"""
from .inputs import CONFIGS, CONFIG_SEEDS, LagaShape, make_inputs  # noqa: F401

__all__ = ["CONFIGS", "CONFIG_SEEDS", "LagaShape", "make_inputs", "laga", "laga_attention", "LagaBlock"]


def __getattr__(name):
    import importlib
    if name == "laga":
        return importlib.import_module(".laga", __name__)
    if name == "laga_attention":          # the differentiable call (torch.autograd plumbing around laga.fwd / laga.bwd)
        return importlib.import_module(".autograd", __name__).laga_attention
    if name == "LagaBlock":               # Algorithm 1 with one rank, every step on the library's kernels
        return importlib.import_module(".block", __name__).LagaBlock
    raise AttributeError(name)
