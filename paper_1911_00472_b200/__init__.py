"""B200 (sm_100a) decoder for Progressive Compressed Records: Python front end of the C ABI."""
from .binding import (ImageInfo, PcrError, pcr_close, pcr_coeffs, pcr_decode, pcr_evict, pcr_get_image,  # noqa: F401
                      pcr_image_blocks, pcr_launch_count, pcr_num_groups, pcr_num_images, pcr_open,
                      pcr_out_bytes, pcr_prefix_bytes, pcr_status, strerror, pcr_get_scan, pcr_set_profiling,
                      pcr_get_profile, pcr_pixels_noalloc, pcr_decode_more, pcr_release_cached_memory, pcr_decode_tensor, pcr_msssim, pcr_msssim_scratch_bytes, pcr_set_upsampling)
from .record import Decoder  # noqa: F401
