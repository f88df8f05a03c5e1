"""B200-native Prioritized Replay Buffer (the Replay Manager + Data Storage of PEARL,
arXiv 2311.09445): a K-ary sum tree over transition priorities with batched insert,
stratified prefix-sum sampling, importance-sampling weights, gather and priority update,
as hand-written CUDA behind a C ABI.  `PrioritizedReplay` is the thin Python binding."""
from .binding import PearlError, PrioritizedReplay, load_library  # noqa: F401

__all__ = ["PrioritizedReplay", "PearlError", "load_library"]
