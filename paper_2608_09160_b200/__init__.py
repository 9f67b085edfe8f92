"""libqknorm: layerwise Query-Key RMSNorm for B200 (sm_100a).

The CUDA library is loaded on first use (see ``binding``); importing this
package never touches it, so the seeded input generators in ``workloads`` can
be used on a machine without the built library.
"""
__all__ = ["workloads", "binding", "build"]
