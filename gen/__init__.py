"""Seeded synthetic inputs shared by the oracle's tests and the CUDA path's tests and bench."""
from .models import SHAPES, LayerShape  # noqa: F401
from .synth import (CONFIGS, CONFIG_ORDER, SynthConfig, SynthLayer, SynthModel,  # noqa: F401
                    draw_activations, draw_weights, make_model, model_sizes, swept_bytes)
