"""The schedule-faithful kernel (thread-block groups play the processes) against the oracle."""
import numpy as np
import pytest
import torch

import paper_1310_4645_b200 as rd
from paper_1310_4645_b200.inputs import make_inputs, WORKLOADS
from oracle import rd_oracle as O
from helpers import oracle_schedule

pytestmark = pytest.mark.gpu

M1 = (2e-6, 1e-10, 5e-11)
SCHEDULES = [("uni_greedy", rd.RD_UNI_GREEDY, rd.RD_PORT_UNI), ("bi_greedy", rd.RD_BI_GREEDY, rd.RD_PORT_BI),
             ("binomial", rd.RD_BINOMIAL, rd.RD_PORT_UNI), ("pipeline_uni", rd.RD_PIPELINE, rd.RD_PORT_UNI),
             ("pipeline_bi", rd.RD_PIPELINE, rd.RD_PORT_BI), ("binary_uni", rd.RD_BINARY, rd.RD_PORT_UNI),
             ("binary_bi", rd.RD_BINARY, rd.RD_PORT_BI), ("butterfly", rd.RD_BUTTERFLY, rd.RD_PORT_BI)]
OPS = {"sum": rd.RD_SUM, "max": rd.RD_MAX, "min": rd.RD_MIN, "prod": rd.RD_PROD}


def run(algo, port, x, seg_bytes, op, rows=None, out=None):
    p, n = x.shape
    h = rd.rd_schedule_create(algo, port, p, 4 * n, seg_bytes, *M1)
    try:
        out = torch.full((n,), 77, dtype=x.dtype, device=x.device) if out is None else out
        st = rd.rd_reduce(h, rows if rows is not None else x, out, OPS[op], exec_mode=rd.RD_EXEC_FAITHFUL,
                          want_stats=True)
        info = rd.rd_schedule_info(h)
        trace = rd.rd_schedule_trace(h) if p > 1 else None
    finally:
        rd.rd_destroy(h)
    ev, off, _ = oracle_schedule(algo, port, p, 4 * n, seg_bytes if seg_bytes else 4 * n, *M1)
    want = O.reduce(ev, x.cpu().numpy().copy(), off, op)
    assert out.cpu().numpy().tobytes() == want.tobytes()
    return st, info, trace


SHAPES = [(8, 4096, 512), (5, 10000, 2500), (13, 3 * 2048 + 36, 2048 + 520), (64, 8192, 1024), (2, 4100, 4100),
          (33, 6000, 1000), (16, 128, 8), (1, 5000, 1000),
          # segments that begin and end at every position inside a 128-bit vector
          (8, 3000, 333), (13, 6180, 999), (4, 64, 3), (32, 8192, 2049), (8, 4099, 1000), (5, 7, 2)]


@pytest.mark.parametrize("name,algo,port", SCHEDULES)
@pytest.mark.parametrize("dist,op", [("int_pm2p20", "sum"), ("normal", "sum"), ("normal", "max"), ("normal", "min"),
                                     ("int_pm2p20", "prod"), ("uniform_pm1", "prod")])
def test_parity_small_shapes(name, algo, port, dist, op):
    for p, n, seg in SHAPES:
        x = make_inputs(p, n, dist, seed=p * 1000 + n, device="cuda")
        if dist == "normal":
            x *= 10.0 ** torch.randint(-4, 5, x.shape, device="cuda", generator=torch.Generator("cuda").manual_seed(1))
        st, info, trace = run(algo, port, x, 4 * seg, op)
        assert st.device_status == 0
        if p > 1:
            assert st.makespan_ns > 0 and st.n_launches == 1
            assert abs(st.predicted_s - info["predicted_seconds"]) < 1e-12
            # every pair was executed: its receiver saw the data and finished after that
            assert (trace[:, 1] >= trace[:, 0]).all() and (trace[:, 2] >= trace[:, 1]).all() and (trace[:, 2] > 0).all()


@pytest.mark.parametrize("name,algo,port", SCHEDULES)
def test_element_path_and_unaligned_buffers(name, algo, port):
    p, n = 8, 3003
    x = make_inputs(p, n, "normal", seed=5, device="cuda")
    run(algo, port, x, 4 * 333, "sum")
    big = make_inputs(p, n + 1, "normal", seed=6, device="cuda")
    rows = [big[i, 1:] for i in range(p)]
    out_big = torch.zeros(n + 1, dtype=torch.float32, device="cuda")
    run(algo, port, big[:, 1:], 4 * 1024, "sum", rows=rows, out=out_big[1:])
    assert out_big[0].item() == 0.0


def test_many_processes_all_resident():
    """1024 processes: one thread block each, all resident at once."""
    p, n = 1024, 2048
    x = make_inputs(p, n, "uniform_pm1", seed=2, device="cuda")
    run(rd.RD_UNI_GREEDY, rd.RD_PORT_UNI, x, 2048, "sum")
    run(rd.RD_BI_GREEDY, rd.RD_PORT_BI, x, 2048, "sum")
    run(rd.RD_BUTTERFLY, rd.RD_PORT_BI, x, 0, "max")


def test_repeated_calls_reuse_flags_and_scratch():
    p, n = 16, 1 << 14
    h = rd.rd_schedule_create(rd.RD_BI_GREEDY, rd.RD_PORT_BI, p, 4 * n, 4096, *M1)
    ev, off, _ = oracle_schedule(rd.RD_BI_GREEDY, rd.RD_PORT_BI, p, 4 * n, 4096, *M1)
    shape = rd.rd_schedule_faithful_shape(h)
    assert shape["blocks_per_process"] >= 1 and shape["slots_per_process"] >= 1
    assert shape["scratch_bytes"] == p * shape["slots_per_process"] * 1024 * 4
    out = torch.empty(n, device="cuda")
    for seed in range(4):
        x = make_inputs(p, n, "normal", seed=seed, device="cuda")
        rd.rd_reduce(h, x, out, rd.RD_SUM, exec_mode=rd.RD_EXEC_FAITHFUL)
        assert out.cpu().numpy().tobytes() == O.reduce(ev, x.cpu().numpy(), off, "sum").tobytes()
    rd.rd_destroy(h)


def test_a_wait_that_runs_out_is_reported_and_the_schedule_stays_usable():
    """With a budget of a microsecond per wait a receiver gives up while its sender is still busy
    with earlier segments: the kernel ends by itself with RD_ERR_TIMEOUT; afterwards the same
    schedule runs to completion."""
    p, n = 8, 1 << 22
    x = make_inputs(p, n, "normal", seed=3, device="cuda")
    out = torch.empty(n, device="cuda")
    h = rd.rd_schedule_create(rd.RD_PIPELINE, rd.RD_PORT_UNI, p, 4 * n, 1 << 20, *M1)
    rd.rd_schedule_set_wait_budget(h, 1e-6)
    with pytest.raises(rd.RdError) as e:
        rd.rd_reduce(h, x, out, rd.RD_SUM, exec_mode=rd.RD_EXEC_FAITHFUL, want_stats=True)
    assert e.value.status == rd.RD_ERR_TIMEOUT
    torch.cuda.synchronize()
    rd.rd_schedule_set_wait_budget(h, 2.0)
    st = rd.rd_reduce(h, x, out, rd.RD_SUM, exec_mode=rd.RD_EXEC_FAITHFUL, want_stats=True)
    assert st.device_status == 0
    ev, off, _ = oracle_schedule(rd.RD_PIPELINE, rd.RD_PORT_UNI, p, 4 * n, 1 << 20, *M1)
    assert out.cpu().numpy().tobytes() == O.reduce(ev, x.cpu().numpy(), off, "sum").tobytes()
    # the tree kernel is unaffected
    rd.rd_reduce(h, x, out, rd.RD_SUM)
    torch.cuda.synchronize()
    assert out.cpu().numpy().tobytes() == O.reduce(ev, x.cpu().numpy(), off, "sum").tobytes()
    rd.rd_destroy(h)


def test_faithful_and_tree_agree_on_config2_and_makespans_are_reported():
    """p = 64, n = 2^20: both execution modes give the same bits for the four schedules of the workload."""
    w = WORKLOADS["config2"]
    model = (w["alpha"], w["beta"], w["gamma"])
    x = make_inputs(w["p"], w["n"], w["dist"], w["seed"], device="cuda")
    a, b = torch.empty(w["n"], device="cuda"), torch.empty(w["n"], device="cuda")
    for algo in (rd.RD_UNI_GREEDY, rd.RD_BINOMIAL, rd.RD_PIPELINE, rd.RD_BINARY):
        h = rd.rd_schedule_create(algo, rd.RD_PORT_UNI, w["p"], 4 * w["n"], w["seg_bytes"], *model)
        rd.rd_reduce(h, x, a, rd.RD_SUM)
        st = rd.rd_reduce(h, x, b, rd.RD_SUM, exec_mode=rd.RD_EXEC_FAITHFUL, want_stats=True)
        rd.rd_destroy(h)
        assert torch.equal(a.view(torch.int32), b.view(torch.int32))
        assert st.makespan_ns > 0


def test_calibration_tool_fits_positive_parameters(capsys):
    """The fitted latency and inverse bandwidth are positive and uni-greedy is the model's favourite."""
    import json
    from paper_1310_4645_b200 import calibrate
    assert calibrate.main(["--p", "8", "--msg-bytes", str(1 << 20)]) == 0
    d = json.loads(capsys.readouterr().out)
    assert d["fitted"]["alpha_s"] > 0 and d["fitted"]["beta_s_per_byte"] > 0
    assert set(d["schedules"]) == {"uni_greedy", "binomial", "pipeline", "binary"}
    assert d["rank_by_model"][0] == "uni_greedy"          # Theorem 5: optimal among in-order one-port schedules
    assert all(v["measured_us"] > 0 for v in d["schedules"].values())
    # the second fit separates the combine from the hand-off (one-port against two-port pipeline periods)
    two = d.get("two_port_fit")
    if two is not None:
        assert two["alpha_s"] > 0 and two["beta_s_per_byte"] >= 0 and two["gamma_s_per_byte"] >= 0
        assert two["beta_s_per_byte"] + two["gamma_s_per_byte"] > 0
        assert two["rank_by_model"][0] == "uni_greedy"


def test_tuning_tool_runs_every_schedule_at_every_power_of_two_segment(tmp_path, capsys):
    """Section VII's procedure on a small case: every schedule, every segment size 2^i, best of a few runs."""
    import json
    from paper_1310_4645_b200 import tune
    out = tmp_path / "tune.jsonl"
    assert tune.main(["--p", "8", "--min-log2-bytes", "16", "--max-log2-bytes", "17", "--reps", "2", "--out", str(out)]) == 0
    rows = [json.loads(ln) for ln in out.read_text().splitlines() if ln.strip()]
    sized = [r for r in rows if "msg_bytes" in r]
    assert {r["msg_bytes"] for r in sized} == {1 << 16, 1 << 17}
    for r in sized:
        assert set(r["schedules"]) == {"uni_greedy", "bi_greedy", "pipeline", "binary", "binomial", "butterfly"}
        for v in r["schedules"].values():
            assert v["best_us"] > 0


def test_randomized_shapes_order_free_results():
    """120 seeded random shapes through the schedule-faithful kernel: int32 sum and max are order free, so
    torch's reductions are an exact reference; lengths and segment sizes ignore every alignment."""
    rng = np.random.default_rng(54321)
    for case in range(120):
        name, algo, port = SCHEDULES[case % len(SCHEDULES)]
        p = int(rng.choice([2, 3, 5, 8, 17, 40, 64, 100, 257]))
        n = int(rng.integers(1, 20000))
        seg = int(rng.integers(1, n + 1)) if rng.random() < 0.5 else int(rng.integers(1, 600))
        x = make_inputs(p, n, "int_pm2p20", seed=case, device="cuda") * int(rng.integers(1, 5000))
        h = rd.rd_schedule_create(algo, port, p, 4 * n, 4 * seg, *M1)
        out = torch.empty(n, dtype=torch.int32, device="cuda")
        try:
            for op, want in ((rd.RD_SUM, x.sum(dim=0, dtype=torch.int64)), (rd.RD_MAX, x.amax(dim=0))):
                out.fill_(-7)
                rd.rd_reduce(h, x, out, op, exec_mode=rd.RD_EXEC_FAITHFUL)
                if op == rd.RD_SUM:
                    want = ((want + (1 << 31)) % (1 << 32) - (1 << 31)).to(torch.int32)
                assert torch.equal(out, want), (case, name, p, n, seg, op)
        finally:
            rd.rd_destroy(h)


def test_eight_byte_elements_in_schedule_faithful_mode():
    """fp64 and int64 through the action lists: whole-vector segments (128-bit accesses) and segments
    that begin 8 bytes into a vector (one element per access)."""
    from helpers import check64, inputs64
    for name, algo, port in SCHEDULES:
        if name == "butterfly":
            continue
        for p, n, seg in ((8, 4096, 512), (13, 3090, 515), (33, 3000, 501), (2, 2050, 2050)):
            check64(algo, port, inputs64(p, n, "normal64", seed=p + n), 8 * seg, "sum", exec_mode=rd.RD_EXEC_FAITHFUL)
            check64(algo, port, inputs64(p, n, "int64", seed=p + n), 8 * seg, "max", exec_mode=rd.RD_EXEC_FAITHFUL)
            check64(algo, port, inputs64(p, n, "near_one", seed=p + n), 8 * seg, "prod", exec_mode=rd.RD_EXEC_FAITHFUL)
    check64(rd.RD_BUTTERFLY, rd.RD_PORT_BI, inputs64(16, 4096, "normal64", seed=3), 0, "sum", exec_mode=rd.RD_EXEC_FAITHFUL)
