"""B200-native continuous speculative decoding hot path (sm_100a CUDA kernels
behind a C ABI).  `inputs` holds the seeded synthetic data generators; `api`
binds the shared library and raises if it is missing (there is no CPU path)."""

__all__ = ["inputs", "api"]
