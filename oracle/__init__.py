"""CPU oracle for the ConfLayers hot path -- TEST INFRASTRUCTURE ONLY.

Only ``tests/``, the smoke check and the benchmark's CPU-baseline / reference leg may import
this package.  It never imports the CUDA package, and the CUDA package never imports it.

Parts:
  * ``conflayers_oracle.c`` -- the Llama-style transformer step with a skip mask and a KV cache,
    the shared-LM-head projection and the entropy confidence (Section 3.1, Eq. 1-4), plain C.
  * ``cycle.py``     -- draft K / verify / greedy-accept loop (Section 3, Figure 2).
  * ``selection.py`` -- adaptive-window skip-set selection (Section 3.2, Eq. 5-10), fp64 Python.
  * ``scoring.py``   -- all-layer confidence scoring and the search-round loop (Sections 3.1, 3.3).
  * ``search.py``    -- generation with the interval-based periodic search (Section 3.3).
"""
from .model import OracleModel, build_oracle, confidence_of_logits, lib  # noqa: F401
from .cycle import (accept_greedy, generate_speculative, generate_vanilla, prefill, speculative_cycle,  # noqa: F401
                    top2_margin)
from .selection import SelectConfig, select_skip_set, selection_details  # noqa: F401
from .scoring import layer_confidences, score_loop  # noqa: F401
from .search import generate_search  # noqa: F401
