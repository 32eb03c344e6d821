"""B200-native TOVA decode step: bounded multi-state attention with eviction.

The product is the CUDA library behind include/tova.h; this package holds its
sources (csrc/), the in-tree build, a ctypes binding with the same names, and
the seeded synthetic workloads.
"""
from .binding import (TOVA_DTYPE_BF16, TOVA_DTYPE_FP32, TOVA_POLICY_H2O_HEAD, TOVA_POLICY_H2O_LAYER, TOVA_POLICY_TOVA,
                      TOVA_POLICY_TOVA_HEAD, TOVA_POLICY_WINDOW, TOVA_POS_AUTO, TovaCache, TovaError, lib, strerror,
                      to_device, tova_cache_bytes, tova_config, tova_decode_step_static)

__all__ = ["TOVA_DTYPE_BF16", "TOVA_DTYPE_FP32", "TOVA_POLICY_H2O_HEAD", "TOVA_POLICY_H2O_LAYER", "TOVA_POLICY_TOVA",
           "TOVA_POLICY_TOVA_HEAD", "TOVA_POLICY_WINDOW", "TOVA_POS_AUTO", "TovaCache", "TovaError", "lib", "strerror",
           "to_device", "tova_cache_bytes", "tova_config", "tova_decode_step_static"]
