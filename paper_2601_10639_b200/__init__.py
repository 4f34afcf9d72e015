"""B200-native STEM FFN layer: y = W_down (SiLU(W_gate x) * E[token_id]), forward and backward.

The compute lives in ``libstem.so`` (hand-written CUDA for sm_100a behind a C ABI, see
``include/stem.h``); :mod:`paper_2601_10639_b200.binding` marshals arguments to it and
:mod:`paper_2601_10639_b200.synth` produces seeded synthetic inputs.  Importing the
package does not load the shared library; the binding does, and raises if it is missing.
"""

__all__ = ["binding", "synth", "build"]
