"""Stacked-LSTM inference forward pass on one B200 (sm_100a): thin Python binding of liblstm_b200.so.

Every step of the computation runs in the library's CUDA kernels; this package only marshals
arguments.  There is no CPU fallback: if the shared library is missing or no CUDA device is usable,
the calls raise.
"""
from .binding import (LSTM, HLSTM, LstmError, hlstm_create, lib_path, load_library, lstm_create, lstm_destroy,  # noqa: F401
                      lstm_forward, lstm_forward_host, lstm_input_projection, lstm_forward_noalloc, lstm_info, lstm_last_error,
                      lstm_probe, lstm_profile_enable, lstm_profile_read, lstm_selftest_timeout, lstm_status,
                      lstm_lhp_points, lstm_nearest_lhp, lstm_fold_input_affine, lstm_csr_lane_layout,
                      LSTM_F32, LSTM_BF16W_F32S, LSTM_DENSE, LSTM_CSR, LSTM_OK, LSTM_ERR_INVALID,
                      LSTM_ERR_UNSUPPORTED, LSTM_ERR_CUDA, LSTM_ERR_NOMEM, LSTM_ERR_TIMEOUT, LSTM_ERR_INTERNAL,
                      LSTM_K_STAGE, LSTM_K_PROJ, LSTM_K_RECUR, LSTM_K_COUNT,
                      LSTM_PROBE_NO_PRODUCTS, LSTM_PROBE_NO_GATES, LSTM_PROBE_NO_EXCHANGE, LSTM_PROBE_WHOLE_STEP)
