"""CPU oracle (test infrastructure): the plain fp64 definition the CUDA library is checked against.

Not part of the product.  Imported only by tests/, the smoke check and the benchmark's CPU-baseline leg.
"""
from .exit_head import (  # noqa: F401
    bf16_decode,
    bf16_rne,
    layer_norm,
    logits,
    softmax_stats,
    exit_decision,
    exit_head,
    compact,
    dssd_accept,
    decisive_rows,
)
from .calibrate import calibrate_threshold, calibrate_threshold_bruteforce, correctness  # noqa: F401,E402
from .cascade import cascade  # noqa: F401,E402
from .dssd_round import dssd_commit, dssd_round, dssd_round_multi  # noqa: F401,E402
from .kl_loss import ce_from_logits, kl_from_logits, kl_to_teacher  # noqa: F401,E402
