"""The library's host-side planner (`wf_plan`, no GPU) against the oracle's row arithmetic and the
paper's shape facts, and the ragged attention work lists against what they must cover."""
import json
import os

import numpy as np
import pytest

from oracle import wf_oracle as O
from paper_2412_11272_b200 import inputs as I
from paper_2412_11272_b200.binding import WfError, wf_plan

ROOT = os.path.dirname(os.path.abspath(__file__))


def _shape(dtype, n_head=4, n_ctx=1536):
    return I.EncoderShape("p", 80, 64 * n_head, 2, n_head, 256, dtype, n_ctx=n_ctx)


def test_token_prefix_sums_match_the_oracle_on_random_batches():
    rng = np.random.default_rng(0)
    for trial in range(50):
        B = int(rng.integers(1, 40))
        H = int(rng.choice([0, 25, 50]))
        lengths = rng.integers(401, 160 * 3000 - 160 * 2 * H, size=B)
        cu, tot, _ = wf_plan(_shape("bf16"), lengths, H, 64, 64 * 1536, int(lengths.sum()))
        frames = [O.n_frames(int(L)) for L in lengths]
        tokens = [O.n_tokens(T + H) for T in frames]
        assert list(np.diff(cu)) == tokens and cu[0] == 0
        assert tot["frames"] == sum(frames) and tot["tokens"] == sum(tokens)
        assert tot["padded_rows"] == sum(2 * (n + 1) for n in tokens)          # one zero row in front, 1-2 behind, even total
        assert tot["front_end_tiles"] == sum((T + 63) // 64 for T in frames)


def test_paper_shape_facts_through_the_planner():
    facts = json.load(open(os.path.join(ROOT, "golden", "paper_shape_facts.json")))
    assert facts                                                               # the fixture that pins the oracle
    cu, tot, _ = wf_plan(_shape("bf16", n_ctx=1500), [30 * 16000], 0, 1, 1500, 30 * 16000)
    assert tot["frames"] == 3000 and list(cu) == [0, 1500]                      # 30 s -> 1500 tokens (Sec. 1.1 / 2.1)
    cu, tot, _ = wf_plan(_shape("bf16"), [16000], 0, 1, 1500, 16000)
    assert tot["frames"] == 100                                                # 1 s -> 100 log-mel rows (Sec. 4.1.2)
    cu, _, _ = wf_plan(_shape("bf16"), [2 * 16000], 50, 1, 1500, 2 * 16000)
    assert list(cu) == [0, 125]                                                # 2.0 s + 50 hush frames -> 125 tokens
    cu, _, _ = wf_plan(_shape("bf16"), [15 * 16000], 0, 1, 1500, 15 * 16000, tail_samples=8000)
    assert list(cu) == [0, 775]                                                # 15 s + 8000-sample hush word -> ~750 tokens (Sec. 4.3.2)
    cu, _, _ = wf_plan(_shape("bf16"), [75, 1], 50, 2, 1500, 0, frames_given=True)
    assert list(cu) == [0, 63, 89]                                             # ceil((75 + 50) / 2), ceil(51 / 2)


def test_planner_status_codes():
    sh = _shape("bf16", n_ctx=100)
    for lengths, kw, status in (([400], {}, "WF_ERR_TOO_SHORT"), ([160 * 300], {}, "WF_ERR_TOO_LONG"),
                                ([16000] * 3, {"max_batch": 2}, "WF_ERR_CAPACITY"),
                                ([16000, 16000], {"max_tokens": 100}, "WF_ERR_CAPACITY"),
                                ([16000, 16000], {"max_samples": 20000}, "WF_ERR_CAPACITY")):
        args = dict(max_batch=8, max_tokens=4096, max_samples=10 ** 7)
        args.update(kw)
        with pytest.raises(WfError) as ei:
            wf_plan(sh, lengths, 50, args["max_batch"], args["max_tokens"], args["max_samples"])
        assert ei.value.status == status, (lengths, kw)
    cu, tot, work = wf_plan(sh, [], 50, 8, 4096, 10 ** 7)                        # an empty batch is legal
    assert list(cu) == [0] and tot["tokens"] == 0 and len(work) == 0


def _covered_bf16(cu, tot, work, n_head):
    """Decodes the bf16 attention work list into a count per (sequence, 128-row tile, head)."""
    E, items = tot["attention_entries"], tot["attention_items"]
    triples, entry_of = work[:3 * E].reshape(E, 3), work[3 * E:]
    assert len(entry_of) == items
    count = {}
    for it in range(items):
        seq, q0k, first = (int(v) for v in triples[entry_of[it]])
        local, kind, q0 = it - first, (q0k & 0xFFFFFFFF) >> 30, q0k & 0x3FFFFFFF
        n = int(cu[seq + 1] - cu[seq])
        if kind == 0:
            cells = [(q0, local), (q0 + 128, local)]
            assert q0 + 128 < n
        elif kind == 1:
            cells = [(q0, 2 * local)] + ([(q0, 2 * local + 1)] if 2 * local + 1 < n_head else [])
        else:
            cells = [(q0, local)]
        for q, h in cells:
            assert q % 128 == 0 and q < n and 0 <= h < n_head
            count[(seq, q // 128, h)] = count.get((seq, q // 128, h), 0) + 1
    return count


@pytest.mark.parametrize("n_head", [4, 5])
def test_bf16_attention_work_list_covers_every_tile_and_head_once(n_head):
    rng = np.random.default_rng(1)
    for trial, (B, hi) in enumerate([(1, 10), (1, 1600), (3, 200), (30, 3000), (64, 1500), (2, 129)]):
        frames = rng.integers(1, hi + 1, size=B)
        cu, tot, work = wf_plan(_shape("bf16", n_head), frames, 50, 64, 64 * 1536, 0, frames_given=True, num_sms=148)
        count = _covered_bf16(cu, tot, work, n_head)
        want = {(i, t, h) for i in range(B) for t in range((int(cu[i + 1] - cu[i]) + 127) // 128) for h in range(n_head)}
        assert set(count) == want and all(v == 1 for v in count.values()), (trial, n_head)
        single = len(want)
        kinds = {(int(v) & 0xFFFFFFFF) >> 30 for v in work[:3 * tot["attention_entries"]].reshape(-1, 3)[:, 1]}
        assert kinds == ({2} if single <= 148 else kinds - {2})                 # single-tile items iff they fit one round of SMs


def test_f32_attention_work_list_is_one_entry_per_16_query_rows():
    frames = [7, 300, 33]
    cu, tot, work = wf_plan(_shape("f32"), frames, 50, 8, 4096, 0, frames_given=True)
    pairs = work.reshape(-1, 2)
    want = [(i, q) for i in range(3) for q in range(0, int(cu[i + 1] - cu[i]), 16)]
    assert sorted(map(tuple, pairs.tolist())) == sorted(want) and tot["attention_entries"] == len(want)
