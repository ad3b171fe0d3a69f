"""B200-native hot path of Astraea's per-step token reduction for video DiTs:
score -> select -> sparse attention -> scatter/reuse, as hand-written sm_100a CUDA
behind a C-ABI library (include/astraea.h).  `binding` marshals arguments only."""

__all__ = ["synth", "accounting", "binding"]
