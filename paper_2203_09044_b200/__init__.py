"""B200-native (sm_100a) CO3 gradient pipeline: error-feedback correction, low-resolution float
conversion, GenNorm-modelled Huffman coding, and parameter-server decode + average.

The compute lives in the CUDA C-ABI library built from csrc/ (see include/co3.h); `binding`
marshals arguments only and raises if the library has not been built.
"""
__all__ = ["binding", "inputs"]
