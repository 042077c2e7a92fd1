"""B200 draft construction for multi-sample speculative decoding.

``synth`` holds the seeded input generators; ``binding`` loads the CUDA
library (``libsdms.so``) and exposes its C entry points.  Nothing here falls
back to a CPU implementation: using the binding without the built library
raises.
"""
