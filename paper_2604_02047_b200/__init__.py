"""B200-native tree-verification step of Goose (tree attention, node top-k, accept walk, KV compaction).

The CUDA library is loaded lazily by :mod:`paper_2604_02047_b200.binding`; importing the
package itself (e.g. for :mod:`paper_2604_02047_b200.synth`) touches no GPU code.
"""

__all__ = ["synth", "binding", "build"]
