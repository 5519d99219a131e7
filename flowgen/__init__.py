"""Seeded synthetic workload generators.

This package only draws random numbers and lays them out in arrays.  It holds
none of the serving path's arithmetic (no feature statistics, no tree walks, no
scores, no model math): anything that depends on such results (the feature
sample that split thresholds are quantiles of) is passed in by the caller.
Both the CUDA library's harness and the CPU oracle's tests draw their inputs
from here, so the two sides see identical bytes.
"""
from .configs import CONFIGS, Config, get_config
from .packets import gen_packets, fast_view, CHUNK_FLOWS, gen_first_packet_headers
from .models import gen_forest, gen_mlp, gen_cnn
from .stream import gen_keys, gen_stream_batch, StreamSource

__all__ = [
    "CONFIGS", "Config", "get_config", "gen_packets", "fast_view", "CHUNK_FLOWS", "gen_first_packet_headers",
    "gen_forest", "gen_mlp", "gen_cnn", "gen_keys", "gen_stream_batch", "StreamSource",
]
