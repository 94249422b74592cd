"""Pins for the paper-mode Token-Table / Task-Table restatement (oracle/task_table.py)
against the one worked example the paper prints (tests/golden/fig3b_task_table.txt)."""
import os

from oracle import task_table as TT

GOLD = os.path.join(os.path.dirname(__file__), "golden", "fig3b_task_table.txt")


def read_golden():
    out = {}
    for line in open(GOLD):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        k, v = line.split(":", 1)
        out[k.strip()] = v.split()
    return out


def fig3b_stages():
    # P with 3 tile blocks at tile size 128 (e.g. 300 tokens), D, V (16-token tree), D
    q_len = [300, 1, 16, 1]
    kv_len = [0, 700, 900, 350]
    return q_len, kv_len


def test_decomposition_matches_fig3b():
    g = read_golden()
    q_len, kv_len = fig3b_stages()
    head_num = 5
    table = TT.token_table(q_len, kv_len, 128)
    assert [e.start for e in table] == [0, 300, 301, 317]
    units = TT.decompose(table, head_num)
    blocks = [len({u.block for u in units if u.stage_id == s}) for s in range(4)]
    assert blocks == [int(x) for x in g["blocks_per_stage"]]
    assert len(units) == int(g["units_per_head"][0]) * head_num


def test_symmetric_round_robin_matches_fig3b():
    g = read_golden()
    C = int(g["num_cores"][0])
    want = [int(x) - 1 for x in g["core_sequence_1based"]]
    assert TT.core_sequence(8, C) == want
    assert TT.core_sequence(16, C) == want + want
    q_len, kv_len = fig3b_stages()
    units = TT.decompose(TT.token_table(q_len, kv_len, 128), 2)
    cores = TT.reorder(units, C)
    # all units placed exactly once
    placed = sorted(u for c in cores for u in c)
    assert placed == sorted(units)
    # each core's list is in non-increasing load; the k-th largest tile sits on core seq[k]
    order = sorted(units, key=lambda u: -u.load)
    seq = TT.core_sequence(len(units), C)
    taken = [0] * C
    for k, u in enumerate(order):
        c = seq[k]
        assert cores[c][taken[c]].load == u.load
        taken[c] += 1


def test_load_is_rows_times_visible_keys():
    units = TT.decompose(TT.token_table([300, 1], [100, 50], 128), 1)
    assert [(u.rows, u.visible) for u in units] == [(128, 228), (128, 356), (44, 400), (1, 51)]
    assert [u.load for u in units] == [128 * 228, 128 * 356, 44 * 400, 51]
    # snake dealing keeps the per-core totals closer than plain round-robin on a sorted list
    loads = sorted(range(1, 17), reverse=True)
    seq = TT.core_sequence(16, 4)
    tot = [0] * 4
    for k, l in enumerate(loads):
        tot[seq[k]] += l
    assert max(tot) - min(tot) == 0
