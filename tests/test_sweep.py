"""The per-operation table driver: its host-side bookkeeping here, a small sweep on the GPU."""
import json

import pytest

from paper_2408_02897_b200 import sweep, workloads


def fake_line(layer, op, fmt, be):
    return json.dumps({"layer": layer, "op": op, "sweep_format": fmt, "role_l": "LHS", "role_r": "RHS",
                       "mean_be": be, "snr_db": 30.0}) + "\n"


def test_resume_bookkeeping_and_summary(tmp_path):
    ops = [o["name"].rsplit("-", 1)[0].split("-", 1)[1]
           for o in workloads.config5_layer(0, "int8", M=256, H=64, F=128, heads=2, S=64)]
    assert len(ops) == 18 and len(set(ops)) == 18
    path = tmp_path / "t.jsonl"
    with open(path, "w") as f:
        for op in ops:
            f.write(fake_line(0, op, "e4m3", 1e-3))
            f.write(fake_line(0, op, "int8", 2e-3))
        for op in ops[:5]:
            f.write(fake_line(1, op, "e4m3", 1e-3))          # layer 1 was interrupted
        f.write('{"layer": 1, "op": "qk')                      # a cut-off line
    assert sweep.finished_layers(str(path), ["e4m3", "int8"]) == {0}
    assert sweep.finished_layers(str(path), ["e4m3", "int8", "e5m2"]) == set()
    assert sweep.finished_layers(str(tmp_path / "none.jsonl"), ["e4m3"]) == set()
    sweep.markdown_table(str(path), str(tmp_path / "t.md"))
    text = open(tmp_path / "t.md").read()
    assert "mean BE e4m3" in text and "| qkv-fwd | LHS | RHS | 1.000e-03 | 30.00 | 2.000e-03 | 30.00 |" in text


def test_roles_follow_the_pass():
    assert workloads.op_roles("L3-ffn1-fwd-e4m3") == ("fwd", "LHS", "RHS")
    assert workloads.op_roles("L3-ffn1-dgrad-e4m3") == ("dgrad", "gradient", "RHS")
    assert workloads.op_roles("L3-ffn1-wgrad-e4m3") == ("wgrad", "LHS", "gradient")
    assert workloads.op_roles("L0-qk-dk-int8") == ("bwd", "gradient", "LHS")
    assert workloads.op_roles("L0-pv-dv-int8") == ("bwd", "LHS", "gradient")


@pytest.mark.gpu
def test_small_sweep_writes_one_line_per_op_and_resumes(tmp_path):
    import oracle
    shape = dict(M=512, H=128, F=256, heads=2, S=128)
    formats = ["e4m3", "int8"]
    rows, ms = sweep.layer_records(1, formats, shape)
    assert len(rows) == 36 and ms > 0
    assert {r["sweep_format"] for r in rows} == set(formats) and all(r["us"] > 0 for r in rows)
    # every line against the oracle's whole-matrix probe of the same op
    tensors = workloads.config5_layer_tensors(1, **shape)
    ops = [o for f in formats for o in workloads.config5_layer(1, f, tensors=tensors, **shape)]
    for o, r in zip(ops, rows):
        L, R = workloads.orient(o)
        want = oracle.derived(oracle.probe(L, R, o["fmt_l"], o["fmt_r"], o["gran_l"], o["gran_r"]))
        for k in ("mean_be", "normwise_be", "rel_l2"):
            assert abs(r[k] - want[k]) <= 1e-4 * want[k], (o["name"], k, r[k], want[k])
        assert abs(10 ** (r["snr_db"] / 10) - 10 ** (want["snr_db"] / 10)) <= 2e-4 * 10 ** (want["snr_db"] / 10)
