"""B200 (sm_100a) integer-only discrete flow inference: thin Python binding over the C ABI in
include/iodf.h. PyTorch supplies device memory and streams; every step of the flow runs in the
library's CUDA kernels. There is no CPU path: loading fails if the library has not been built."""
from .binding import (IodfError, Model, iodf_create, iodf_destroy, iodf_forward, iodf_inverse,
                      iodf_inverse_level, IODF_LEVEL_PRIOR, IODF_LEVEL_COUPLINGS, IODF_PLAN_LATENCY,
                      IODF_PLAN_THROUGHPUT, iodf_forward_patches,
                      iodf_inverse_patches, Codec, iodf_codec_create, iodf_rans_encode, iodf_rans_decode_block,
                      iodf_codec_check, iodf_rans_packed_capacity, iodf_rans_pack, iodf_rans_unpack,
                      iodf_compress_host, iodf_decompress_host,
                      iodf_forward_host, iodf_inverse_host, iodf_forward_timed, iodf_inverse_timed,
                      iodf_get_layout, iodf_forward_static, iodf_static_scratch_bytes_per_image,
                      IODF_STATIC_SCRATCH_BYTES, iodf_check, iodf_strerror,
                      iodf_launches_per_call, iodf_selftest_timeout, iodf_int8_mma_peak, iodf_level_kernel_name,
                      iodf_level_images_per_cta,
                      load_library,
                      DECLARED_SYMBOLS)

__all__ = ["IodfError", "Model", "iodf_create", "iodf_destroy", "iodf_forward", "iodf_inverse",
           "iodf_inverse_level", "IODF_LEVEL_PRIOR", "IODF_LEVEL_COUPLINGS", "IODF_PLAN_LATENCY",
           "IODF_PLAN_THROUGHPUT", "iodf_forward_patches",
           "iodf_inverse_patches", "Codec", "iodf_codec_create", "iodf_rans_encode", "iodf_rans_decode_block",
           "iodf_codec_check", "iodf_rans_packed_capacity", "iodf_rans_pack", "iodf_rans_unpack",
           "iodf_compress_host", "iodf_decompress_host",
           "iodf_forward_host", "iodf_inverse_host", "iodf_forward_timed", "iodf_inverse_timed", "iodf_get_layout", "iodf_forward_static", "iodf_static_scratch_bytes_per_image",
           "IODF_STATIC_SCRATCH_BYTES", "iodf_check", "iodf_strerror",
           "iodf_launches_per_call", "iodf_selftest_timeout", "iodf_int8_mma_peak", "iodf_level_kernel_name",
           "iodf_level_images_per_cta",
           "load_library",
           "DECLARED_SYMBOLS"]
