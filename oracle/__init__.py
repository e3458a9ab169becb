"""fp64 CPU oracle for prompt-sharing tree attention (test infrastructure only).

Nothing in the product path may import this package: it exists so that the
CUDA kernels can be checked against a plain, slow, obviously correct
restatement of the paper's definitions.  It shares no code with the kernels.
"""
