"""B200-native hot path of continuous depth batching (CDB) for looped language models.

`binding` wraps the C-ABI library (libcdb.so, hand-written sm_100a CUDA); importing it fails
loudly when the library has not been built.  `synth` holds the seeded synthetic input
generators (data only, none of the method's arithmetic).  `engine` is the thin host-side
driver that feeds row descriptors to the library.
"""

__all__ = ["binding", "synth", "engine"]
