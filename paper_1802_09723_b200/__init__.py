"""B200 (sm_100a) Recurrent Residual Module library: thin Python binding over the C ABI.

Every step of the hot path runs in the CUDA kernels of librrm_b200.so; this package only
marshals arguments.  Importing it does not load the shared library; the first call does,
and fails loudly if the library is missing or cannot be built.
"""
from .binding import (RRMError, LayerDesc, Stats, Options, Net, Layer, lib, desc_from_spec, net_from_specs,
                      layer_from_spec, fc_step_noalloc, aecs_predict, measure_alu_peak, KIND, DTYPE, ACT, VARIANT)

__all__ = ["RRMError", "LayerDesc", "Stats", "Options", "Net", "Layer", "lib", "desc_from_spec", "net_from_specs",
           "layer_from_spec", "fc_step_noalloc", "aecs_predict", "measure_alu_peak", "KIND", "DTYPE", "ACT", "VARIANT"]
