"""Crystal-KV decode hot path for NVIDIA B200: thin Python binding over the C-ABI library."""
from .binding import (CrystalKV, CrystalKVError, Config, load_library, declared_symbols,  # noqa: F401
                      THINK, ANSWER, EVICT, FULLKV)
