"""B200-native per-stream phrase boosting inside batched Transducer decoding.

``binding`` holds the Python side of the C-ABI library (argument marshalling only);
``workloads`` holds the seeded synthetic input generators.  Nothing is imported eagerly so
that the input generators can be used without the CUDA library being built.
"""
