"""Seeded synthetic inputs for the multi-LoRA / multi-stream / DS2D decode path.

This package only *prepares inputs*: model shapes, random weight draws, the
INT4 group quantiser that produces the packed weight blobs, adapter draws,
prompts and draft-tree shapes.  It contains none of the arithmetic of the
decode step itself (no dequantisation, no projections, no attention, no
acceptance rule), so both the CPU oracle and the CUDA path can consume the
same blobs without sharing any implementation.
"""
from .configs import ModelCfg, CFG0, CFG1, CFG2, CFG3, PROJ_NAMES, proj_shape, PROJ_BITS
from .synth import (quantize_int4, quantize_int4_per_channel, pack_nibbles, make_model, make_adapter,
                    make_prompt_ids, make_hidden, build_tree, tree_depths, ds2d_template, make_forecast,
                    make_candidates, SynthModel)

__all__ = ["ModelCfg", "CFG0", "CFG1", "CFG2", "CFG3", "PROJ_NAMES", "PROJ_BITS", "proj_shape",
           "quantize_int4", "quantize_int4_per_channel", "pack_nibbles", "make_model", "make_adapter",
           "make_prompt_ids", "make_hidden", "build_tree", "tree_depths", "ds2d_template", "make_forecast",
           "make_candidates", "SynthModel"]
