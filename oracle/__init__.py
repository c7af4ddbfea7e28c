"""CPU oracle for the convolution forward path.  Test infrastructure only: imported by
tests/, by the smoke check and by the bench's CPU-baseline leg, never by the product."""
from .conv_oracle import (  # noqa: F401
    ConvParams,
    batchnorm,
    bn_fold,
    build,
    cast_f32_to_f16,
    conv_fast,
    conv_naive,
    conv_points,
    double_to_half_bits,
    half_bits_to_double,
    inner_product,
    num_threads,
    out_dim,
    nchw_to_nhwc,
    nhwc_to_nchw,
    repack_weights,
)
