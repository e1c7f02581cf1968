"""B200-native selective-KV hot path: score -> top-k select -> gather-pack -> two-source sparse decode.

The public calls (`sg_score`, `sg_select_topk`, `sg_pack_kv`, `sg_sparse_decode_attn`, ...) live in
`paper_2607_28150_b200.binding`, a thin ctypes layer over the C-ABI library `libsmartgen.so`
(hand-written sm_100a CUDA).  They are re-exported here lazily so that the input generators in
`paper_2607_28150_b200.workloads` and the build step in `paper_2607_28150_b200.build` can be
imported before the library exists.  There is no fallback: touching any `sg_*` name without the
built library raises.
"""
import importlib

__all__ = ["binding", "workloads", "build"]


def __getattr__(name):
    if name in ("binding", "workloads", "build", "pipeline", "replicas"):
        return importlib.import_module(__name__ + "." + name)
    if name.startswith("sg_") or name.startswith("SG_") or name in ("Shape", "SmartGenError"):
        return getattr(importlib.import_module(__name__ + ".binding"), name)
    raise AttributeError(name)
