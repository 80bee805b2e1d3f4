"""B200-native forward pass of a ViT pipeline stage: CUDA kernels behind a C boundary
(include/vit.h) and a ctypes binding with the same entry-point names."""
from .binding import *  # noqa: F401,F403
from .binding import VitModel, VitConfig, VitError, make_config, lib, LIB_PATH, EXPORTS  # noqa: F401
