"""fp64 CPU oracle of the LSTM forward pass: test infrastructure only.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this package; the
CUDA library and its Python binding never do, and this package never imports them.
"""
from .lstm_oracle import build, forward, forward_hlstm, input_projection, threads, dense_to_csr  # noqa: F401
