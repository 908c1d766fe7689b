"""pdkv: block-free transfer of paged KVCache on one B200 (sm_100a).

``binding``   ctypes binding over ``libpdkv.so`` with the names of ``include/pdkv.h``
``session``   convenience holder of the C handles of one batch
``workloads`` seeded synthetic inputs (no transfer arithmetic)
``build``     builds the shared library with nvcc
``p2d``       sender rank / receiver rank protocol over ``torch.distributed``

Nothing here falls back to a CPU path: without the built library every call
raises.
"""
__all__ = ["binding", "session", "workloads", "build", "p2d"]
