"""B200-native DiLoCo outer step (standard / naive delayed / eager) and inner AdamW.

The work is done by hand-written sm_100a CUDA kernels behind the C ABI declared in
``include/diloco.h`` (built in-tree as ``libdiloco.so``).  ``binding`` is a thin ctypes
layer with the same names; ``inputs`` draws the seeded synthetic workloads; ``worker`` is the
one-replica-per-GPU deployment form (state + asynchronous all-reduce ring).  There is no
CPU fallback: calling into the binding without the built library raises.
"""
__all__ = ["binding", "inputs", "worker"]
