"""Host logic of the freezing-frequency schedule (Section 3.2: the frozen set is updated once
per f processed samples)."""
from paper_2411_11038_b200.network import FreezeSchedule


def _selection_steps(f, batch, steps):
    s = FreezeSchedule(f, batch)
    out = []
    for i in range(steps):
        if s.due():
            out.append(i)
            s.selected()
        s.advance()
    return out, s


def test_every_step_when_f_not_above_batch():
    steps, s = _selection_steps(16, 24, 5)
    assert steps == [0, 1, 2, 3, 4] and s.selections == 5 and s.steps == 5


def test_once_per_f_samples():
    # f = 4096 samples at 24 samples per step: 171 steps reach 4104 >= 4096
    steps, _ = _selection_steps(4096, 24, 400)
    assert steps == [0, 171, 342]
    steps, _ = _selection_steps(16384, 128, 300)
    assert steps == [0, 128, 256]


def test_first_step_always_selects():
    s = FreezeSchedule(10 ** 9, 1)
    assert s.due()
    s.selected()
    s.advance()
    assert not s.due()
