"""B200-native hot path of the Orthrus generation step (dual-view block attention,
exact consensus, KV commit).  `workloads` draws the seeded synthetic inputs;
`binding` wraps the C-ABI CUDA library and raises if it has not been built."""

__all__ = ["workloads", "binding"]
