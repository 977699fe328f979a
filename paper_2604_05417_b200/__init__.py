"""MetaSD draft-verify hot path for NVIDIA B200: C-ABI CUDA library + thin Python binding."""
from .binding import (BF16, FP32, UCB, DUCB, SWUCB, REWARD_BD, REWARD_BE, PATH_AUTO, PATH_STREAMING,
                      PATH_FUSED, MetaSD, MetasdError, VerifyResult, load_library, pointer_table)

__all__ = ["BF16", "FP32", "UCB", "DUCB", "SWUCB", "REWARD_BD", "REWARD_BE", "PATH_AUTO",
           "PATH_STREAMING", "PATH_FUSED", "MetaSD", "MetasdError", "VerifyResult", "load_library",
           "pointer_table"]
