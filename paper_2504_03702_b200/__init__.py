"""B200-native load anticipator and load-aware router (PreServe, arXiv 2504.03702, Sec. 4.3).

`binding` is the thin ctypes layer over the C-ABI library (include/preserve_b200.h);
`state.DeviceState` holds the device tensors those calls act on; `workloads` draws the
seeded synthetic inputs.  The CUDA library is loaded when `binding` is imported and there
is no fallback of any kind.
"""
__all__ = ["binding", "state", "workloads", "build"]
