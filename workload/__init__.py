"""Seeded synthetic workloads shared by the oracle tests and the CUDA harness."""
from .generator import *  # noqa: F401,F403
from .generator import (WORKLOADS, ModelShape, Workload, TINY, LLAMA2_7B, LLAMA2_13B, LLAMA2_70B,  # noqa: F401
                        normal_fp16, token_ids, weight_tensor, layer_weights, shard_weights,
                        prompt_ids, forced_decode_ids, weight_seed, tensor_shape,
                        standard_normal_f32, stream_key)
