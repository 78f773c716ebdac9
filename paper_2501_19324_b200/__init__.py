"""B200-native (sm_100a) step loop of Reward-Guided Speculative Decoding behind a C-ABI library.

`binding` marshals arguments to librsd.so; nothing here computes on the CPU."""
from .binding import (Engine, Model, RsdError, lib, EXPORTS, RSD_F32, RSD_BF16, RSD_DRAFT, RSD_PRM, RSD_TARGET,
                      RSD_HEAD_LM, RSD_HEAD_REWARD_SIGMOID, RSD_HEAD_REWARD_RAW, RSD_DEBUG_KEEP_LOGITS, RSD_DEBUG_NO_GRAPHS, RSD_DEBUG_PERSISTENT_DECODE, RSD_DEBUG_MEGA_PROFILE)

__all__ = ["Engine", "Model", "RsdError", "lib", "EXPORTS"]
