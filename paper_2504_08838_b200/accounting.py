"""Accounting around the sparse drafter: MAC counts, the improvement factor, greedy speculative decoding.

Plain host-side arithmetic (no device code): the quantities the paper uses to turn a drafter's
quality (mean accepted length, MAL) and cost (MACs or latency) into an end-to-end figure.

* MACs per token of a drafter (Section "MACs analysis"): the decoder-block linears, of which a
  fine-grained-sparse drafter executes only the kept fraction, plus the LM head, which stays
  dense (Section "Results": only the decoder blocks are pruned).  Embedding look-ups and the
  attention score products are not counted; with that convention a 50 %-sparse
  Llama-3.2-3B-shaped drafter needs 43.87 % fewer MACs than the dense one (Abstract).
* Improvement factor (Eq. 3): MAL / (k c + 1) with k draft tokens per round and c the cost of one
  drafter forward pass relative to one target forward pass (latency ratio, or MAC ratio for the
  theoretical variant).
* Greedy draft-then-verify (Eq. 1 and Eq. 2): the drafter proposes k tokens, each the argmax of
  its own distribution; the target checks them in order, keeps a draft token while it equals its
  own argmax, and at the first mismatch (or after k matches) contributes one token of its own.
  A round therefore yields (accepted drafts + 1) tokens, which is what MAL averages (footnote of
  Eq. 3), and the text produced is exactly the target's own greedy text.
"""

from __future__ import annotations

from typing import Callable, List, Sequence, Tuple

from .synth import DrafterShape

LLAMA3_VOCAB = 128256      # Llama-3 tokenizer (not stated in the paper; reproduces its 43.87 %)


def decoder_macs_per_token(shape: DrafterShape) -> int:
    """Multiply-accumulates of all decoder-block linears (q, k, v, o, gate, up, down) for one token."""
    return shape.blocks * shape.block_macs()


def drafter_macs_per_token(shape: DrafterShape, vocab: int, sparsity: float = 0.0) -> float:
    """MACs of one forward pass for one token: kept decoder-linear weights plus the dense LM head."""
    if not 0.0 <= sparsity <= 1.0:
        raise ValueError("sparsity must lie in [0, 1]")
    return (1.0 - sparsity) * decoder_macs_per_token(shape) + shape.hidden * vocab


def mac_reduction(shape: DrafterShape, vocab: int, sparsity: float) -> float:
    """Fraction of the dense drafter's MACs that a drafter of the given decoder sparsity saves."""
    dense = drafter_macs_per_token(shape, vocab, 0.0)
    return (dense - drafter_macs_per_token(shape, vocab, sparsity)) / dense


def improvement_factor(mal: float, k: int, c: float) -> float:
    """Eq. 3: expected speed-up of speculative decoding over sampling from the target alone."""
    if k < 1 or c < 0.0 or mal < 1.0:
        raise ValueError("need k >= 1, c >= 0 and MAL >= 1 (every round yields the target's token)")
    return mal / (k * c + 1.0)


NextToken = Callable[[Sequence[int]], int]     # greedy model: context -> argmax token


def speculative_decode(draft_next: NextToken, target_next: NextToken, prompt: Sequence[int], k: int,
                       max_new_tokens: int, eos: int | None = None) -> Tuple[List[int], List[int]]:
    """Greedy draft-then-verify.  Returns (generated tokens, tokens gained in each round).

    `draft_next` and `target_next` map a token context to that model's argmax next token (Eq. 1:
    drafts are argmax tokens of the drafter; Eq. 2: a draft survives iff it is the target's argmax,
    else the target's token replaces it and the round ends).  A real target scores the k + 1
    positions of a round in one forward pass; calling `target_next` position by position computes
    the same tokens.  Generation stops after `max_new_tokens` tokens or at `eos`.
    """
    if k < 1:
        raise ValueError("k >= 1 draft tokens per round")
    out: List[int] = []
    rounds: List[int] = []
    ctx = list(prompt)
    while len(out) < max_new_tokens and (eos is None or not out or out[-1] != eos):
        drafts, dctx = [], list(ctx)
        for _ in range(k):
            t = draft_next(dctx)
            drafts.append(t)
            dctx.append(t)
        gained = 0
        for j in range(k + 1):
            want = target_next(ctx)
            ctx.append(want)                      # the token kept at this position is always the target's argmax
            out.append(want)
            gained += 1
            stop = len(out) >= max_new_tokens or (eos is not None and want == eos)
            if stop or j == k or drafts[j] != want:
                break
        rounds.append(gained)
    return out, rounds


def mean_accepted_length(rounds: Sequence[int]) -> float:
    """MAL: tokens gained per round, accepted drafts plus the target's one, averaged over rounds."""
    if not rounds:
        raise ValueError("no rounds")
    return sum(rounds) / float(len(rounds))
