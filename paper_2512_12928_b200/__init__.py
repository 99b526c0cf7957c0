"""ps-kvswap: B200-native KV-block swap and paged decode attention (after ProServe, Section 4.3).

`paper_2512_12928_b200.workloads` draws seeded synthetic inputs and is importable anywhere.
`paper_2512_12928_b200.binding` loads the CUDA library and raises if it has not been built.
"""
__all__ = ["workloads", "binding"]
