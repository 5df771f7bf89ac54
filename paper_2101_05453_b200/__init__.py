"""Integer-only quantized LSTM forward pass for NVIDIA B200: Python binding of libqlstm.so."""
from .binding import (BiQLSTM, ERR_ARG, ERR_CUDA, ERR_DIM, ERR_LAUNCH, ERR_NOMEM, ERR_RANGE, ERR_TIMEOUT, IMPL_AUTO,  # noqa: F401
                      IMPL_FAST, IMPL_SIMPLE, OK, QLSTM, QlstmError, lib, library_path, strerror)
