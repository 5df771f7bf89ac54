"""CPU oracle of the integer-only LSTM forward pass.  TEST INFRASTRUCTURE ONLY.

Imported by tests, the smoke check and the benchmark's CPU-baseline leg; never by the
CUDA package.  `qlstm_ref` wraps the plain-C oracle, `qlstm_np` is an independent
pure-Python restatement for tiny cases.
"""
