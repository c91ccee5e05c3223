"""B200-native sparse decode attention for Pre-hoc Sparsity (PrHS / CIS).

The product is the CUDA library built from `csrc/` (C ABI declared in `include/prhs.h`);
`binding` marshals arguments into it and nothing else.  Importing the package does not
load the library; the first use of `binding` does, and raises if it has not been built.
"""
__all__ = ["binding", "workloads", "build"]
