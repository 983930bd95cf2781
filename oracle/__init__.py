"""fp64 CPU oracle for ONNX Conv, Gemm and the two pooling operators.  Test infrastructure only.

Only the test-suite, the smoke check and the CPU-baseline legs of the benchmark
may import this package; the product library never does, and this package never
imports the product.
"""
from .reference import (  # noqa: F401
    OracleShapeError,
    build,
    conv2d,
    conv2d_output_shape,
    gemm,
    gemm_c_strides,
    threads,
)
from .pooling import (  # noqa: F401
    PoolShapeError,
    global_average_pool,
    maxpool2d,
    maxpool2d_output_shape,
)
