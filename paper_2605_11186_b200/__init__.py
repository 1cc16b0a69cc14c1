"""B200-native tree-verification forward for CATS-style self-speculative decoding.

``paper_2605_11186_b200.binding`` loads the CUDA library (``libcats.so``) and
exposes the C-ABI entry points; ``paper_2605_11186_b200.inputs`` holds the
seeded synthetic-input generators.  Nothing is imported eagerly here so that
the input generators can be used without the CUDA library.
"""
__version__ = "0.1.0"
