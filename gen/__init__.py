"""Seeded synthetic input generators (no method arithmetic lives here)."""
from .inputs import (activations, calibration_batch, weights, outlier_channels,
                     bf16_bits, from_bf16_bits)

__all__ = ["activations", "calibration_batch", "weights", "outlier_channels",
           "bf16_bits", "from_bf16_bits"]
