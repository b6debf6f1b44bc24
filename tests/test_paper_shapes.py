"""The paper-shaped workloads against the values the paper prints (App. A.2, architecture table;
fixture tests/golden/paper_architectures.txt), and the printed group widths against the width
rule of Sec. 3.1, Eq. 1."""
import os

import pytest

import oracle as O
from paper_2604_23108_b200.inputs import WORKLOADS

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_architectures.txt")


def _rows():
    out = {}
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        f = line.split()
        if f[0] == "alpha":
            out["alpha"] = {f[1]: float(f[2]), f[3]: float(f[4])}
            continue
        out[f[0]] = dict(d=int(f[1]), N_g=int(f[2]), K_g=int(f[3]), N_e=int(f[4]), K_e=int(f[5]),
                         N_s=int(f[6]), widths=tuple(int(v) for v in f[7:]))
    return out


@pytest.mark.parametrize("scale,name", [("3B", "paper_3b_layer"), ("14B", "paper_14b_layer")])
def test_paper_shaped_workloads_use_the_printed_architecture(scale, name):
    row, wl = _rows()[scale], WORKLOADS[name]
    assert wl.d_model == row["d"]
    assert wl.n_groups == row["N_g"] and wl.k_groups == row["K_g"]
    assert wl.n_experts == row["N_e"] and wl.experts_per_group == row["N_e"] // row["N_g"]
    assert wl.k_experts == row["K_e"]
    assert tuple(wl.group_width) == row["widths"]
    assert wl.T % 4096 == 0                      # whole sequences of the paper's length


@pytest.mark.parametrize("scale", ["1B", "3B", "14B"])
def test_printed_group_widths_follow_eq_1(scale):
    """Eq. 1 mirrors the widths around a base width: W_i + W_{N_g+1-i} = 2 W_base for every i
    (1-based), and the widths increase with i."""
    row = _rows()[scale]
    w = row["widths"]
    assert len(w) == row["N_g"] and list(w) == sorted(w)
    sums = {w[i] + w[len(w) - 1 - i] for i in range(len(w))}
    assert len(sums) == 1
    w_base = sums.pop() / 2
    assert w[0] < w_base < w[-1]


@pytest.mark.parametrize("scale", ["1B", "3B", "14B"])
def test_oracle_accepts_the_printed_architectures(scale):
    row = _rows()[scale]
    cfg = O.OracleConfig(d_model=row["d"], n_groups=row["N_g"], experts_per_group=row["N_e"] // row["N_g"],
                         k_groups=row["K_g"], k_experts=row["K_e"], group_width=list(row["widths"]))
    assert cfg.n_experts == row["N_e"]
    assert row["K_e"] <= row["K_g"] * (row["N_e"] // row["N_g"])     # Eq. 5 can always pick K_e experts


def test_default_loss_coefficients_are_the_papers_best_row():
    a = _rows()["alpha"]
    from paper_2604_23108_b200 import binding as B
    ocfg = O.OracleConfig(d_model=8, n_groups=1, experts_per_group=1, k_groups=1, k_experts=1, group_width=[8])
    gcfg = B.Config(d_model=8, n_groups=1, experts_per_group=1, k_groups=1, k_experts=1, group_width=[8])
    assert (ocfg.alpha_e, ocfg.alpha_g) == (a["alpha_E"], a["alpha_G"])
    assert (gcfg.alpha_e, gcfg.alpha_g) == (a["alpha_E"], a["alpha_G"])
