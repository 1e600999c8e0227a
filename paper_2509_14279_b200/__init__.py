"""rkv: bulk verification of candidate-kernel outputs on B200 (sm_100a).

``population`` (seeded synthetic candidates) imports without the CUDA library;
``binding`` loads ``librkv.so`` on first use and raises if it is missing.
"""
__version__ = "0.1.0"
