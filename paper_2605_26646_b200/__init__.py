"""B200-native hot path of a multi-agent PPO update: role-level advantages, grouped LM-head
log-prob / entropy, and the PPO-clip + KL loss with its backward, behind the C ABI of libunity.so.

``binding`` mirrors the C entry points (argument marshalling only); ``workloads`` draws seeded
synthetic inputs; ``build`` compiles the CUDA sources in-tree.  Importing the package does not load
the shared library; the first call into ``binding`` does, and fails loudly if it cannot.
"""
from . import workloads  # noqa: F401

__all__ = ["binding", "build", "sharding", "workloads"]
