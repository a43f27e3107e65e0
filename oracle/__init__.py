"""CPU fp64 oracle for memory-augmented sliding-window (MASW) speculative decoding.

TEST INFRASTRUCTURE ONLY.  This package is a plain, slow, obviously-correct restatement of what the
paper defines (Section 4 "Method": Eq. 3 and the local-window definition, the projection equations of
"Projection and KV materialization", the "Memory update cycle", Section 4.3, and the standard
accept/reject rule of Section 3.1; the masked prefill pass of Section 4.3 and Appendix C).  It shares no code with the CUDA library and never imports it.
Only the tests, the smoke check and the benchmark's ``cpu_baseline`` / ``--impl reference`` legs may
import it; the product path never does.

Parity status: every function here is pinned by the CPU tests (hand-computed example, closed forms,
library cross-checks, invariants, brute force).  The one thing that stays "parity unpinned" is the
*quality* of the learned compression (whether a slot preserves acceptance): it depends on trained
adaptor weights, which are out of scope.
"""
from .bf16 import bf16_bits_to_f64, f64_to_bf16_bits, round_to_bf16  # noqa: F401
from .attend import attend, attend_chunked  # noqa: F401
from .memory import DraftMemory, rope_rotate, memory_entries_closed_form  # noqa: F401
from .verify import verify_attend  # noqa: F401
from .prefill import prefill_attend, n_prefill_slots  # noqa: F401
from .accept_reject import accept_reject, spec_exp, integer_weights  # noqa: F401
from .speedup import sd_speedup, tokens_per_second  # noqa: F401
from .fp8 import dequantize_e4m3, e4m3_to_f64, fp16_round  # noqa: F401
