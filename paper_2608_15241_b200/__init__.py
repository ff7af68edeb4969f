"""B200-native mixed-adapter LoRA linear layer (sm_100a CUDA behind a C ABI).

`paper_2608_15241_b200.binding` is the thin Python layer over the C-ABI shared library;
`paper_2608_15241_b200.workloads` draws the seeded synthetic inputs.  Importing the package
loads nothing native; the library is loaded (and must exist) on first use of the binding.
"""
__all__ = ["binding", "workloads", "build"]
