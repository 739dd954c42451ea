"""CPU oracle for the LAQ hot path -- test infrastructure only.

Only ``tests/``, ``__graft_entry__.smoke()`` and the CPU-baseline / ``--impl reference`` legs of
``bench.py`` may import this package.  It shares nothing with the CUDA library.
"""
from .binding import (  # noqa: F401
    MODEL_LOGREG_BIN, MODEL_SOFTMAX, MODEL_MLP2, MODEL_SYNTH, MODEL_GIVEN,
    FLAG_QUANT_OFF, FLAG_TRIGGER_OFF,
    build, lib, quantize, decode, pack_codes, unpack_codes, trigger, batch_offset,
    grad_logreg_bin, grad_softmax, grad_mlp2, synth_gradient, round_bf16, lyapunov, OracleLaq,
)
