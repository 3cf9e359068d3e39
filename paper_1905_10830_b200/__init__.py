"""B200-native feature-map transform codec (arXiv 1905.10830): thin Python binding of the
C-ABI library in `csrc/` (declared in `include/tc.h`).  The binding only marshals arguments;
every step of the coding path runs in the library's CUDA kernels.  torch is used for device
memory and streams only."""
from .binding import (  # noqa: F401
    TcError, Context, Model, Codebook, EncodedStream, StreamLayout, Stats,
    tc_create, tc_fit_pca, tc_model_import, tc_model_export, tc_build_codebook,
    tc_codebook_import, tc_codebook_export, tc_encode_bound, tc_encode, tc_encode_noalloc, tc_encode_many, tc_decode_many, tc_roundtrip_host, tc_decode, tc_stats,
    tc_fit_state_create, tc_fit_state_update, tc_fit_state_export, tc_fit_state_import, tc_fit_state_finish, FitState,
    tc_fold_forward, tc_fold_inverse,
    tc_get_status, tc_force_exact_path, tc_last_path, tc_host_huffman_lengths, tc_host_eigh, tc_device_eigh, TC_EIG_DEVICE, TC_EIG_HOST, library_path, load_library,
)
from .pipeline import CodedLayer, calibrate_layer_by_layer, run_chain, code_layer  # noqa: F401,E402
