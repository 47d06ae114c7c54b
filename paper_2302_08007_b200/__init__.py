"""B200-native BDR / MX quantization library (Python side: argument marshalling only).

The compute lives in the CUDA C-ABI library under ``csrc/``; ``binding`` loads it lazily and fails
loudly if it is missing.  ``synth`` holds the seeded input generators (no method arithmetic).
"""
