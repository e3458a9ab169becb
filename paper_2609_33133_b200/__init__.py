"""Prompt-sharing tree attention (prefill + replay, forward + backward) for B200 (sm_100a).

The compute lives in the C-ABI library built from csrc/ (see include/augtree.h);
`binding` marshals arguments to it and nothing else.  Importing `binding`
raises if the library has not been built: there is no CPU fallback.
"""
__all__ = ["workloads"]
