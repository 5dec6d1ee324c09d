"""Seeded synthetic inputs for Generalized PolyDot coded matmul / coded DNN runs.

This package holds only input recipes: shapes, splits, node counts, seeds and the
random matrices themselves.  It contains none of the method's arithmetic (no
encoding, thresholds, decoding or error location), so that both the CPU oracle
and the CUDA library can be fed from it without sharing any of their own code.
"""

from .configs import (  # noqa: F401
    CodedMatmulConfig,
    MLPConfig,
    AutoencoderConfig,
    CONFIG_1_TINY,
    CONFIG_2_MATVEC,
    CONFIG_3_MATMUL,
    CONFIG_4_MLP,
    CONFIG_5_AUTOENCODER,
    matmul_inputs,
    mlp_inputs,
    autoencoder_inputs,
    scaled_down,
)
