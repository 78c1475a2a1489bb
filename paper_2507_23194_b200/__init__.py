"""B200-native batched candidate-vs-reference output verifier (the data-parallel hot path of the
GEAK Evaluator's functionality test). ``gv`` is the binding of the C ABI; ``workloads`` holds the
seeded synthetic inputs; ``build`` compiles the CUDA library in-tree."""
__all__ = ["gv", "workloads", "build"]
