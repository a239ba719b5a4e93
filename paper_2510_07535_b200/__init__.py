"""B200-native verification step of long-context speculative decoding (OWL / HOWL):
tree-masked split-KV attention of drafted tokens against a paged bf16 KV cache and greedy tree
acceptance, as hand-written sm_100a CUDA kernels behind the C ABI of ``include/owlverify.h``.

``binding`` marshals torch tensors into that ABI; ``workloads`` draws seeded synthetic inputs;
``build`` compiles the library.  Nothing here computes on the CPU.
"""
from . import workloads  # noqa: F401
from .binding import (OwlContext, OwlDims, OwlError, load_library, make_dims, owl_howl_route,  # noqa: F401
                      owl_tree_accept_static, status_string)
