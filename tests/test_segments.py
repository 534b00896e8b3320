"""Algorithm 1 bookkeeping (host logic, no GPU): a scripted rollout engine and hand-worked pool contents."""
import numpy as np
import pytest

from paper_2507_19766_b200.segments import Sample, SegmentRollout, pack_experience


class ScriptedEngine:
    """Each sample has a scripted total length (None = never ends); tokens are 100*prompt + position and
    the log-prob of a token is -(version + 1) so the producing version can be read back from it."""

    def __init__(self, total_len):
        self.total_len = total_len
        self.calls = []

    def __call__(self, samples, max_len, version):
        self.calls.append((version, [(s.prompt_id, s.response_id, len(s)) for s in samples], max_len))
        out = []
        for s in samples:
            total = self.total_len[(s.prompt_id, s.response_id)]
            left = max_len if total is None else min(max_len, total - len(s))
            toks = [100 * s.prompt_id + len(s) + k for k in range(left)]
            eos = total is not None and len(s) + left == total
            out.append((toks, [-(version + 1.0)] * left, eos))
        return out


def test_three_termination_conditions_and_versions():
    # global max 12 in 3 segments of 4.  Lengths: (0,0) ends at 3 (step 0); (0,1) ends at 6 (step 1);
    # (1,0) never ends -> truncated at 12 (step 3, it joined at step 1); (1,1) ends at exactly 4.
    eng = ScriptedEngine({(0, 0): 3, (0, 1): 6, (1, 0): None, (1, 1): 4})
    r = SegmentRollout(global_max_seq_len=12, max_segment_count=3)
    assert r.each_segment_length == 4

    r.step(eng, new_prompts=[0], samples_per_prompt=2, version=0)
    assert [(s.prompt_id, s.response_id) for s in r.experience_pool] == [(0, 0)]
    assert [(s.prompt_id, s.response_id, len(s)) for s in r.unfinished_pool] == [(0, 1, 4)]
    exp0 = r.take_experience()
    assert exp0[0].finished and not exp0[0].truncated and exp0[0].segment_version == [0, 0, 0]
    assert r.experience_pool == []

    r.step(eng, new_prompts=[1], samples_per_prompt=2, version=1)
    # the unfinished sample is rolled out first, continued from its 4 tokens
    assert eng.calls[1][1] == [(0, 1, 4), (1, 0, 0), (1, 1, 0)]
    exp1 = {(s.prompt_id, s.response_id): s for s in r.take_experience()}
    assert set(exp1) == {(0, 1), (1, 1)}
    s01 = exp1[(0, 1)]
    assert s01.tokens == [0, 1, 2, 3, 4, 5] and s01.segment_version == [0, 0, 0, 0, 1, 1]
    assert s01.old_logp == [-1.0] * 4 + [-2.0] * 2 and s01.n_segments == 2
    assert exp1[(1, 1)].finished and len(exp1[(1, 1)]) == 4        # EOS on the segment's last token: complete
    assert [(s.prompt_id, s.response_id, len(s)) for s in r.unfinished_pool] == [(1, 0, 4)]

    r.step(eng, new_prompts=[], samples_per_prompt=2, version=2)
    assert r.experience_pool == [] and len(r.unfinished_pool[0]) == 8
    r.step(eng, new_prompts=[], samples_per_prompt=2, version=3)
    (s10,) = r.take_experience()
    assert s10.truncated and not s10.finished and len(s10) == 12 and s10.n_segments == 3
    assert s10.segment_version == [1] * 4 + [2] * 4 + [3] * 4
    assert r.unfinished_pool == []


def test_pack_experience_layout():
    a = Sample(0, 0, tokens=[5, 6, 7], old_logp=[-1, -1, -2], segment_version=[3, 3, 4])
    e = Sample(0, 1)                                    # no tokens: skipped
    b = Sample(1, 0, tokens=[9, 8], old_logp=[-0.5, -0.25], segment_version=[4, 4])
    p = pack_experience([a, e, b], advantages=[1.5, 7.0, -0.5])
    assert p["seq_offsets"].tolist() == [0, 3, 5] and p["seq_offsets"].dtype == np.int32
    assert p["targets"].tolist() == [5, 6, 7, 9, 8]
    assert p["old_logp"].tolist() == [-1, -1, -2, -0.5, -0.25] and p["old_logp"].dtype == np.float32
    assert p["segment_version"].tolist() == [3, 3, 4, 4, 4]
    assert p["advantages"].tolist() == [1.5, -0.5] and p["current_version"] == 4
    q = pack_experience([], [])
    assert q["seq_offsets"].tolist() == [0] and q["targets"].size == 0


def test_rejects_bad_engine_and_bad_config():
    with pytest.raises(ValueError):
        SegmentRollout(10, 3)
    r = SegmentRollout(8, 2)
    with pytest.raises(ValueError):
        r.step(lambda s, m, v: [([1] * 5, [0.0] * 5, False)], [0], 1, 0)      # 5 tokens in a 4-token segment
    with pytest.raises(ValueError):
        r.step(lambda s, m, v: [], [0], 1, 0)


def test_balance_into_calls():
    from paper_2507_19766_b200.segments import balance_into_calls
    lengths = [100, 10, 10, 10, 60, 40, 30, 20, 20]            # 300 tokens
    calls = balance_into_calls(lengths, 150)
    assert sorted(i for c in calls for i in c) == list(range(9))            # a partition
    loads = [sum(lengths[i] for i in c) for c in calls]
    assert len(calls) == 2 and loads == [150, 150]
    assert all(c == sorted(c) for c in calls)
    # long tail: capacity forces three calls; each within capacity, spread no worse than the largest sample
    rng = np.random.default_rng(5)
    lengths = np.minimum(131072, (2048 * rng.pareto(1.2, size=200) + 256).astype(np.int64)).tolist()
    calls = balance_into_calls(lengths, 131072)
    loads = [sum(lengths[i] for i in c) for c in calls]
    assert sorted(i for c in calls for i in c) == list(range(200))
    assert max(loads) <= 131072 and len(calls) >= -(-sum(lengths) // 131072)
    assert max(loads) - min(loads) <= max(lengths)
    assert balance_into_calls([], 10) == []
    with pytest.raises(ValueError):
        balance_into_calls([11], 10)
