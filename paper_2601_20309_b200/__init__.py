"""B200-native KV-block rotation engine (swap-out / swap-in / full-duplex rotate).

The CUDA library is loaded lazily by ``paper_2601_20309_b200.binding``; importing the
package alone (for example to reach the seeded workload generators) loads nothing.
"""
__all__ = ["binding", "workload", "build"]
