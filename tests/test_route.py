"""Three-stage routing, traffic accounting (Section 3.2 of the paper): the plan's slabs placed on
nodes must carry exactly the volumes the paper claims -- trainers send one model copy, every rollout
node receives exactly its de-duplicated volume over RDMA -- and give the lower bound of Eq. 1."""
import numpy as np

from paper_2609_25442_b200 import binding as wb
from wb_workloads import WB_BF16, Layout, make_workload


def plan_of(tl, rl):
    return wb.Plan(wb.Layout(tl.tensors, tl.slices), wb.Layout(rl.tensors, rl.slices))


def test_figure_example_tp2_trainer_dp4_rollout():
    """The worked example of the three-stage figure: trainer TP2 (T0, T1), rollouts DP4 (R0-R3) on two
    nodes of two workers.  Every rollout needs the whole model, yet each receives a distinct quarter
    from the trainers, then the nodes swap what they received, then the workers of a node share."""
    rows, cols = 8, 4096
    tl, rl = Layout("t"), Layout("r")
    for t in range(2):                                  # TP2: row halves
        k = tl.add_tensor(f"T{t}", t, WB_BF16, rows // 2 * cols)
        tl.add_slice(k, 0, cols, 1, 0, rows, cols, t * rows // 2, 0, rows // 2, cols)
    for r in range(4):                                  # DP4: four full replicas
        k = rl.add_tensor(f"R{r}", r, WB_BF16, rows * cols)
        rl.add_slice(k, 0, cols, 1, 0, rows, cols, 0, 0, rows, cols)
    tl.freeze(); rl.freeze()
    plan = plan_of(tl, rl)
    plan.verify()
    M = rows * cols * 2
    st, ingress, required = wb.wb_route_account(plan, [0, 0], [1, 1, 2, 2], 3, trainer_gbs=400.0, node_gbs=400.0)
    assert st["model_bytes"] == M == plan.stats()["src_bytes_read"]
    assert st["receive_bytes"] == M                     # trainers collectively send one copy
    assert st["max_trainer_rank_egress"] == M // 2      # balanced over the TP ranks
    assert [plan.rank_bytes(1, r) for r in range(4)] == [M // 4] * 4    # a distinct quarter each
    assert st["external_bytes"] == M                    # each node gets the other node's half once
    assert list(ingress) == [0, M, M] and list(required) == [0, M, M]   # RDMA ingress == M_v per node
    assert st["internal_bytes"] == 2 * M                # per node: each worker copies its peer's half
    assert st["direct_rdma_bytes"] == 4 * M             # direct all-to-all: every worker pulls a full copy
    assert st["max_rollout_rank_rdma_ingress"] == M // 2
    assert abs(st["t_min_seconds"] - M / 400e9) < 1e-15   # Eq. 1: max(M/B_T, M_v/B_v)


def test_eq1_picks_the_slower_of_trainer_egress_and_node_ingress():
    wl = make_workload("cfg3", "small")
    plan = plan_of(wl.trainer, wl.rollout)
    M = wl.ckpt_numel() * 2
    # trainer: PP stage 0 on node 0, stage 1 on node 1; both rollout TP ranks on node 2
    tn = [0, 0, 0, 0, 1, 1, 1, 1]
    st, ingress, required = wb.wb_route_account(plan, tn, [2, 2], 3, trainer_gbs=800.0, node_gbs=100.0)
    assert st["model_bytes"] == st["receive_bytes"] == M
    assert st["external_bytes"] == 0                    # one rollout node: nothing to exchange over RDMA
    H, L = wl.meta["spec"].H, wl.meta["spec"].L
    assert st["internal_bytes"] == (2 * L + 1) * H * 2  # the norms, shared inside the node
    assert list(ingress) == [0, 0, M] and list(required) == [0, 0, M]
    assert abs(st["t_min_seconds"] - M / 100e9) < 1e-12
    st2, _, _ = wb.wb_route_account(plan, tn, [2, 2], 3, trainer_gbs=50.0, node_gbs=100.0)
    assert abs(st2["t_min_seconds"] - M / 50e9) < 1e-12
    # both TP ranks on different nodes: the norms cross once more, everything else stays put
    st3, ingress3, required3 = wb.wb_route_account(plan, tn, [2, 3], 4)
    assert st3["external_bytes"] == (2 * L + 1) * H * 2 and st3["internal_bytes"] == 0
    assert list(ingress3) == list(required3)
    assert int(required3[2]) + int(required3[3]) == M + (2 * L + 1) * H * 2


def test_unreplicated_models_need_no_exchange():
    wl = make_workload("cfg4", "small")
    plan = plan_of(wl.trainer, wl.rollout)
    M = wl.ckpt_numel() * 2
    st, ingress, required = wb.wb_route_account(plan, list(range(8)), [8], 9)
    assert st["receive_bytes"] == st["direct_rdma_bytes"] == M
    assert st["external_bytes"] == st["internal_bytes"] == 0
    assert int(ingress[8]) == int(required[8]) == M
    assert sum(plan.rank_bytes(0, r) for r in range(8)) == M      # source dtype == destination dtype here
