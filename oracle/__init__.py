"""CPU oracle for the tree-verification step (TEST INFRASTRUCTURE, not product code).

A plain, slow, fp64 restatement of what the target model's verification step computes
in EAGLE-2-style speculative decoding as the paper uses it (Section 3.1: the target
verifies the drafted tokens in one forward pass and incorrect tokens are discarded;
Section 4.1: tree attention, top-k 10, 60 tokens; abstract / Section 4.1: decoding is
lossless with respect to the target).

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this
package. It shares no code with the CUDA library and never calls it. Every function is
pinned by tests that do not restate its own formula (closed forms, brute force on tiny
inputs, special cases that reduce to a separately written textbook routine, invariants);
no function here is "parity unpinned".
"""

from .tree import tree_depth, tree_mask_bits, tree_positions, is_valid_tree  # noqa: F401
from .rope import rope_rotate_half  # noqa: F401
from .attention import (  # noqa: F401
    bf16_bits_to_f64,
    f64_to_bf16_bits,
    tree_attn,
    causal_attn_textbook,
)
from .accept import (  # noqa: F401
    vocab_argmax,
    accept_topdown,
    accept_bruteforce,
    kv_compact,
)
from .sample import accept_sample, decision_margins, softmax_f64  # noqa: F401
from .draft_tree import rerank_tree, topk_logprob  # noqa: F401
from .compress import visual_pool, visual_prune  # noqa: F401
