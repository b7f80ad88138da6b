"""CPU oracle package: TEST INFRASTRUCTURE ONLY.

Holds (1) ``conv_oracle.c`` -- the plain definition of valid-mode 1-D / 2-D
convolution (Eq. 2 and Eq. 3 of the paper) in fp64 / exact int32, reached from
Python through ctypes, ``stencil_oracle.c`` -- the iterated 3x3 stencil with fixed boundary values (the second
workload), and (2) ``systolic_sim.py`` -- a design-faithful CPU
simulator of the paper's linear systolic arrays (Section 2, Section 4 Code 2-4,
Table 2) that pins the *method*.

Nothing here is imported by the product package; the product never falls back
to this code.  It shares no code with the CUDA path.
"""
from .conv import (  # noqa: F401
    build_oracle,
    conv1d_f32,
    conv1d_f32_strided,
    conv1d_f32_taps_outer,
    conv2d_f32_strided,
    conv1d_f32_at,
    conv2d_f32,
    conv2d_f32_taps_outer,
    conv2d_f32_at,
    conv1d_u8s8_s32,
    conv2d_u8s8_s32,
    conv2d_u8s8_i64,
    num_threads,
    set_num_threads,
    stencil2d_f32,
)
