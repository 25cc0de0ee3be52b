"""CPU oracle for the partial-token GRPO policy-gradient step (NAT).

TEST INFRASTRUCTURE ONLY.  This package is the slow, plain fp64 statement of
what the CUDA library must compute.  It is imported by the tests, by the
smoke check and by the benchmark's CPU-baseline leg; the product package never
imports it and shares no code, table or constant generator with it.

Parity status of each function (what pins it to something other than itself):

  philox4x32_10     pinned: known-answer vectors of the published generator,
                    and an independent big-integer restatement in the tests.
  grpo_adv          pinned: z-score closed form for binary rewards, numpy
                    mean/std cross-check, zero-sum invariant.
  select            pinned: the paper's closed forms for the survival
                    probabilities, E[L], exact enumeration of every cut value
                    in rational arithmetic, binomial frequency test for URS.
  select_survival   pinned: boundary values of the 24-bit draw against the exact count
                    ceil(p 2^24), the uniform-cutoff schedule reproducing the uniform law,
                    prefix structure, and exhaustive enumeration of a geometric cut law
                    showing the HT estimator unbiased (Proposition 1).
  select_cutlaw     pinned: the three properties of Eq. rpc-survival (pi_1 = 1, monotone,
                    positive where the law has mass), pi against the suffix sums of q in
                    rational arithmetic, the uniform law reproducing the uniform-cutoff
                    closed form bit for bit, draw boundaries against the exact integer
                    count, cut frequencies over seeds, and exhaustive enumeration of the
                    cuts showing the HT estimator unbiased (Proposition 1).
  compact           pinned: brute-force list comprehension, segment structure
                    for prefix modes.
  gather/scatter    pinned: numpy fancy indexing, scatter(gather(x)) = mask * x, and the
                    packed prefixes being the per-response slices [cu_i, cu_i + L_i).
  policy_loss_fwd   pinned: softmax rows sum to one, scipy log_softmax,
                    old_logp == logp closed form, p = 1 full-token GRPO written
                    as an independent double loop, exhaustive enumeration of
                    masks / cuts (Proposition 1); the optional KL term by its closed form.
  policy_loss_bwd   pinned: central finite differences of policy_loss_fwd,
                    zero column sums, exhaustive enumeration of the gradient's
                    expectation, saturated-clip zero gradient.
  policy_loss_dW_rows  pinned: equals the corresponding rows of policy_loss_bwd's dW (itself
                    pinned by finite differences) and central differences on the chosen rows.
"""
from .philox import philox4x32_10  # noqa: F401
from .nat_oracle import (  # noqa: F401
    SEL_URS,
    SEL_RPC,
    SEL_DET,
    grpo_adv,
    select,
    select_survival,
    select_cutlaw,
    cutlaw_counts,
    compact,
    gather_rows,
    scatter_rows,
    policy_loss_fwd,
    policy_loss_bwd,
    policy_loss_dW_rows,
    grad_coeff,
)
