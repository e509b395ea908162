"""BitLinear forward of BitNet b1.58 as sm_100a CUDA kernels behind a C-ABI library.

The Python layer only marshals arguments (torch tensors -> device pointers);
every step of the path runs in the CUDA library.  Importing the package is
cheap; the shared library is loaded on first use and its absence is an error.
"""
