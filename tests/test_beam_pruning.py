"""Beam-pruning state machine (Sec. 4.2.2): the Python oracle against hand-worked cases, and the
library's C implementation against the oracle, bit for bit, on synthetic token streams with
injected misalignment, punctuation noise and substitutions (no GPU involved)."""
import numpy as np

from oracle import beam_oracle as BO
from paper_2412_11272_b200 import inputs as I

VOCAB = 200
SPECIAL = set(range(0, 20))          # ids 0..19 stand for punctuation / timestamps / special tokens


def _flags():
    f = np.zeros(VOCAB, np.uint8)
    f[list(SPECIAL)] = 1
    return f


# ----- oracle pins: cases worked by hand from the paper's three mechanisms ------------------------

def test_identical_transcript_keeps_beam_one():
    ref = [50, 51, 52, 53, 54]
    beams, idx, fb = BO.run_session(ref, SPECIAL, ref)
    assert beams == [1, 1, 1, 1, 1] and idx == 5 and not fb


def test_alignment_skips_a_trimmed_prefix_and_leading_special_tokens():
    ref = [40, 41, 50, 51, 52, 53]                        # the buffer was trimmed: decoding now starts at 50
    beams, idx, fb = BO.run_session(ref, SPECIAL, [3, 50, 51, 7, 52, 53])   # 3 = timestamp, 7 = punctuation
    assert beams == [1] * 6 and idx == 6 and not fb


def test_alignment_failure_and_mismatch_trigger_fallback_for_good():
    beams, idx, fb = BO.run_session([50, 51, 52], SPECIAL, [99, 50, 51])
    assert beams == [1, 5, 5] and fb and idx is None        # search found nothing
    beams, idx, fb = BO.run_session([50, 51, 52, 53], SPECIAL, [50, 51, 60, 53, 5])
    assert beams == [1, 1, 1, 5, 5] and fb and idx == 2     # 60 != 52: full beam from the next round on


def test_new_content_beyond_the_reference_needs_the_full_beam():
    beams, idx, fb = BO.run_session([50, 51], SPECIAL, [50, 51, 4, 70, 71])
    assert beams == [1, 1, 1, 1, 5] and fb                   # special token 4 is free, 70 has no reference


def test_first_match_is_taken_when_the_token_repeats():
    p = BO.BeamPruner([50, 60, 50, 61], SPECIAL)
    assert p.step(50) == 1 and p.i == 1
    assert p.step(60) == 1 and p.step(50) == 1 and p.step(61) == 1 and p.i == 4


def test_special_tokens_inside_the_reference_are_passed_over():
    # the previous transcript "50 , 51 <ts> 52" against "50 , 51 52": the comma and the timestamp of
    # the reference are no comparison targets, so 51 meets 51 and 52 meets 52
    beams, idx, fb = BO.run_session([50, 7, 51, 3, 52], SPECIAL, [50, 7, 51, 52])
    assert beams == [1, 1, 1, 1] and idx == 5 and not fb
    # punctuation on one side only, either side
    beams, idx, fb = BO.run_session([50, 7, 51, 52], SPECIAL, [50, 51, 9, 52])
    assert beams == [1, 1, 1, 1] and idx == 4 and not fb
    # a real mismatch behind a reference comma still falls back, and the index stays behind the last match
    beams, idx, fb = BO.run_session([50, 7, 51], SPECIAL, [50, 60, 51])
    assert beams == [1, 1, 5] and fb and idx == 1
    # a reference that ends in punctuation is exhausted for a new word
    beams, idx, fb = BO.run_session([50, 7], SPECIAL, [50, 70])
    assert beams == [1, 1] and fb and idx == 1


# ----- the library against the oracle ----------------------------------------------------------------

def _stream(seed, n):
    u = I.uniform01(seed, 77, n)
    return [int(20 + v * (VOCAB - 20)) for v in u]


def test_library_matches_oracle_on_synthetic_sessions():
    from paper_2412_11272_b200.binding import BeamPruner
    flags = _flags()
    n_cases, reduced, rounds = 0, 0, 0
    for seed in range(200):
        prev = _stream(seed, 40)
        u = I.uniform01(seed, 78, 200)
        if seed % 2:                                        # previous transcripts carry punctuation / timestamps too
            v = I.uniform01(seed, 79, 80)
            prev = [t for k, t in enumerate(prev) for t in ([int(v[40 + k] * 20)] if v[k] < 0.2 else []) + [t]]
        cut = int(u[0] * 10)                                # audio trimmed at the front
        cur = prev[cut:] + _stream(seed + 1000, 8)          # and new audio appended at the end
        out = []
        for k, tok in enumerate(cur):
            if u[1 + k] < 0.15:
                out.append(int(u[60 + k] * 20))             # inserted punctuation / timestamp token
            if u[100 + k] < (0.02 if seed % 3 else 0.0):
                tok = int(20 + u[140 + k] * (VOCAB - 20))   # substitution
            out.append(tok)
        if seed % 17 == 0:
            out = [199, 198] + out                          # alignment cannot succeed
        want, idx, fb = BO.run_session(prev, SPECIAL, out)
        p = BeamPruner(prev, flags)
        got, nxt = [], 1
        for tok in out:
            got.append(nxt)
            nxt = p.step(tok)
        st = p.state()
        assert got == want, seed
        assert st["fallen_back"] == fb and st["reference_index"] == (-1 if idx is None else idx)
        assert st["rounds"] == len(out)
        p.close()
        n_cases += 1
        reduced += sum(1 for b in got if b == 1)
        rounds += len(got)
    assert n_cases == 200 and 0.3 < reduced / rounds < 1.0


def test_library_rejects_bad_arguments():
    from paper_2412_11272_b200.binding import BeamPruner, WfError
    import pytest
    with pytest.raises(WfError):
        BeamPruner([VOCAB + 5], _flags())                   # reference id outside the vocabulary
    p = BeamPruner([50], _flags())
    with pytest.raises(WfError):
        p.step(VOCAB)
    p.close()
