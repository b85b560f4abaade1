"""B200-native tree-causal prefix-shared attention (forward and backward).

The compute path lives in the C-ABI shared library built from `csrc/`
(`libpsrl.so`); `binding` marshals arguments to it and nothing else.  There is
no CPU or PyTorch fallback: using the binding without the built library raises.
"""
__all__ = ["binding", "workloads", "build"]
