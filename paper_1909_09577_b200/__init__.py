"""B200 (sm_100a) time-channel separable convolution block: thin Python binding over the C ABI."""
from .binding import (  # noqa: F401
    Context, EncoderSpec, block_desc, sepconv_workspace_bytes, sepconv_fwd, sepconv_fwd_static, sepconv_bwd,
    encoder_workspace_bytes, encoder_fwd_bwd, sepconv_infer, encoder_infer, load_library, strerror, SepconvError,
)
