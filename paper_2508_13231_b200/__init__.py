"""libkvp: KV-cache placement scoring and bound search on one B200 (CUDA, sm_100a).

`paper_2508_13231_b200.kvp` is the thin binding over the C ABI of include/kvp.h;
`paper_2508_13231_b200.workloads` names the synthetic configurations. Importing
this package loads nothing; the shared library is opened on first use of `kvp`
and the import fails loudly when it has not been built.
"""
__all__ = ["kvp", "workloads"]
