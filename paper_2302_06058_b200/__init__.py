"""Bi-Mask per-layer sparse training step on one B200: a C-ABI CUDA library (libbimask.so,
declared in include/bimask.h) and this thin binding.  The library is loaded on first use."""
from .binding import *  # noqa: F401,F403
from .binding import (BimaskError, LayerArgs, ConvArgs, TrainArgs, alloc_layer_buffers, lib, make_conv_args, make_layer_args,
                      make_train_args)  # noqa: F401
