"""B200-native speculative-step attention for Sparrow (verification and text-anchored window
modes).  The product is the C-ABI library built from ``csrc/``; ``binding`` marshals arguments to
it and ``workloads`` builds seeded synthetic inputs.  Nothing here computes attention on the CPU.
"""
__all__ = ["binding", "workloads", "build"]
