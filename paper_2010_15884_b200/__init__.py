"""Warp-level software systolic convolution for NVIDIA B200 (sm_100a).

1-D and 2-D valid-mode convolution (correlation form, Eq. 2 and Eq. 3 of
"Systolic Computing on GPUs for Productive Performance") executed as linear
software systolic arrays on the 32 lanes of a warp, in weight-stationary (BSM),
output-stationary (FBS) and input-stationary (SBM) projections.

The compute lives in ``libsysconv.so`` (CUDA, C ABI, see ``include/sysconv.h``);
``binding`` is a thin ctypes layer over it.  There is no CPU fallback: every
call fails loudly when the library is missing.  ``inputs`` only draws the
seeded synthetic workloads.
"""

_BINDING_NAMES = (
    "sysconv1d", "sysconv2d", "sysconv1d_strided", "sysconv2d_strided", "sysconv1d_host", "sysconv2d_host",
    "sysconv1d_host_static", "static_scratch_bytes", "conv1d", "conv2d", "spacetime_describe", "sysconv1d_spacetime", "sysconv2d_separable", "conv2d_separable", "sysconv1d_host_multi", "host_multi_workspace_bytes",
    "load_library", "library_path", "SysconvError", "WS", "OS", "IS", "FSM", "BFS", "FFS", "F32", "U8S8_S32",
    "DESIGN_NAMES", "status_string", "design_name", "version", "host_workspace_bytes",
    "launch_count", "device_status",
)


def __getattr__(name):
    if name in _BINDING_NAMES:
        from . import binding
        return getattr(binding, name)
    raise AttributeError(name)
