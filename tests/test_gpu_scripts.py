"""The measurement scripts of the package run (small sizes; they print JSON lines)."""
import json

import pytest

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gpu():
    import torch
    from paper_2604_16957_b200 import tq
    assert torch.cuda.is_available()
    return tq, torch


def test_ablation_script_runs_and_orders_sanely(gpu, capsys):
    from paper_2604_16957_b200 import ablation
    ablation.run(1024, 11, 1.0, 0)
    rows = [json.loads(line) for line in capsys.readouterr().out.splitlines() if line.startswith("{")]
    by = {r["variant"]: r for r in rows}
    assert by["fp16 K, fp16 V"]["cosine_min"] == 1.0
    for name in ("int4 K, fp16 V", "fp16 K, int4 V", "int4 K, int4 V"):
        assert 0.98 < by[name]["cosine_mean"] < 1.0
    assert by["int4 K, int4 V"]["cosine_mean"] <= max(by["int4 K, fp16 V"]["cosine_mean"], by["fp16 K, int4 V"]["cosine_mean"])


def test_workload_script_runs_one_small_workload(gpu, capsys):
    from paper_2604_16957_b200 import workloads
    workloads.decode_workload("probe", 1, 8, 2, 128, 2048, 128 ** -0.5, 2, 1, True, window=512, S_q=2, page_tokens=64)
    row = json.loads(capsys.readouterr().out.strip().splitlines()[-1])
    assert row["us_per_call"] > 0 and row["page_tokens"] == 64 and row["S_q"] == 2
