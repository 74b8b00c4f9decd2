"""MAC counts, the improvement factor (Eq. 3) and greedy draft-then-verify (Eq. 1, Eq. 2): CPU only.

Pins: the values the paper prints (tests/golden/paper_printed_values.txt), hand-counted rounds,
and the property that strict top-1 verification reproduces the target's own greedy text.
"""

import os

import pytest

from paper_2504_08838_b200 import accounting as acc
from paper_2504_08838_b200 import synth


def _golden():
    path = os.path.join(os.path.dirname(__file__), "golden", "paper_printed_values.txt")
    out = {}
    for line in open(path):
        line = line.strip()
        if line and not line.startswith("#"):
            k, v = line.split()
            out[k] = float(v)
    return out


def test_mac_reduction_of_the_50_percent_llama3b_drafter_is_the_printed_one():
    g = _golden()
    r = acc.mac_reduction(synth.LLAMA_3B, acc.LLAMA3_VOCAB, 0.5)
    assert abs(100.0 * r - g["mac_reduction_percent_llama3b_50"]) < 0.005
    assert acc.decoder_macs_per_token(synth.LLAMA_3B) == 2_818_572_288
    # nothing pruned, nothing saved; everything pruned leaves the dense LM head
    assert acc.mac_reduction(synth.LLAMA_3B, acc.LLAMA3_VOCAB, 0.0) == 0.0
    assert acc.drafter_macs_per_token(synth.LLAMA_3B, acc.LLAMA3_VOCAB, 1.0) == 3072 * acc.LLAMA3_VOCAB


def test_improvement_factor_is_eq3():
    g = _golden()
    # a free drafter (c = 0) gains MAL tokens per target pass; a drafter as slow as the target
    # (c = 1) pays k + 1 passes per round
    assert acc.improvement_factor(g["mal_llama3b_sd2_50"], 5, 0.0) == g["mal_llama3b_sd2_50"]
    assert acc.improvement_factor(4.0, 3, 1.0) == 1.0
    assert abs(acc.improvement_factor(4.16, 4, 0.05) - 4.16 / 1.2) < 1e-12
    # at equal k and c the printed MALs order the drafters as the abstract says: SD^2 / layer-pruned = 1.59
    ratio = acc.improvement_factor(g["mal_llama3b_sd2_50"], 4, 0.1) / acc.improvement_factor(g["mal_llama3b_layer_pruned_50"], 4, 0.1)
    assert abs(ratio - g["mal_ratio_sd2_over_layer_pruned"]) < 0.005
    with pytest.raises(ValueError):
        acc.improvement_factor(0.5, 4, 0.1)


def _table_model(table, default):
    """Greedy model given by a look-up on the last token."""
    return lambda ctx: table.get(ctx[-1], default)


def test_hand_counted_rounds():
    # target continues 1 -> 2 -> 3 -> 4 -> 5 -> 6 -> 7 ...; the drafter agrees except after 3 (says 9)
    target = _table_model({i: i + 1 for i in range(20)}, 0)
    draft = _table_model({**{i: i + 1 for i in range(20)}, 3: 9}, 0)
    out, rounds = acc.speculative_decode(draft, target, [1], k=3, max_new_tokens=6)
    # first draft-verify cycle: drafts 2, 3, 9 -> 2 and 3 accepted, 9 rejected and replaced by the target's 4: 3 tokens
    # second cycle: context ends in 4: drafts 5, 6, 7 all accepted, the target adds 8: 4 tokens (cut at 6 in total)
    assert out == [2, 3, 4, 5, 6, 7]
    assert rounds == [3, 3]
    out, rounds = acc.speculative_decode(draft, target, [1], k=3, max_new_tokens=7)
    assert out == [2, 3, 4, 5, 6, 7, 8] and rounds == [3, 4]
    assert acc.mean_accepted_length(rounds) == 3.5
    # a drafter that is always wrong still gains the target's token every round: MAL = 1
    wrong = lambda ctx: 99
    out, rounds = acc.speculative_decode(wrong, target, [1], k=4, max_new_tokens=5)
    assert out == [2, 3, 4, 5, 6] and rounds == [1] * 5 and acc.mean_accepted_length(rounds) == 1.0
    # a perfect drafter gains k + 1 per round
    out, rounds = acc.speculative_decode(target, target, [1], k=4, max_new_tokens=10)
    assert rounds == [5, 5] and acc.mean_accepted_length(rounds) == 5.0


def test_output_is_the_targets_own_greedy_text():
    # strict top-1 verification: whatever the drafter proposes, the text is the target's (Section
    # "Speculative decoding"); models here depend on the last two tokens, drawn from a seeded stream
    V = 7
    for seed in range(20):
        u = synth.uniform(1234 + seed, 2 * V * V)
        tt = {(a, b): int(u[a * V + b] * V) for a in range(V) for b in range(V)}
        dd = {(a, b): int(u[V * V + a * V + b] * V) if u[a * V + b] < 0.4 else tt[(a, b)] for a in range(V) for b in range(V)}
        target = lambda ctx, t=tt: t[(ctx[-2], ctx[-1])]
        draft = lambda ctx, d=dd: d[(ctx[-2], ctx[-1])]
        ref, ctx = [], [1, 2]
        for _ in range(40):
            ref.append(target(ctx))
            ctx.append(ref[-1])
        for k in (1, 2, 5):
            out, rounds = acc.speculative_decode(draft, target, [1, 2], k=k, max_new_tokens=40)
            assert out == ref
            assert sum(rounds) == 40 and all(1 <= r <= k + 1 for r in rounds)


def test_eos_ends_generation():
    target = _table_model({1: 2, 2: 3, 3: 0}, 0)
    out, rounds = acc.speculative_decode(target, target, [1], k=5, max_new_tokens=50, eos=0)
    assert out == [2, 3, 0] and rounds == [3]
