"""Host side of the generic taskflow front end (Section 4.2: split propagation -- Algorithm 1 --, Task Descriptors;
Section 4.3: events with static thresholds, queue order).  No GPU: the compiler is host code of the library."""
import pytest

from paper_2605_23764_b200 import binding as B

SW, ADD, NONE = B.MOE_TF_SWIGLU, B.MOE_TF_ADD, B.MOE_TF_NO_EVENT


def _pair(M=100, C=64, rows_a=8, rows_b=8, add_split=((0, 0),)):
    # tensors: 0 = x [M,2C], 1 = s [M,C], 2 = r [M,C], 3 = z [M,C]
    tensors = [(M, 2 * C), (M, C), (M, C), (M, C)]
    ops = [B.tf_operator(SW, [0], [1], rows_a, split_inputs=None),
           B.tf_operator(ADD, [1, 2], [3], rows_b, split_inputs=list(add_split))]
    return tensors, ops


def _simulate(plan, workers):
    """Workers take descriptors in queue order and block on their dependent event: the queue must drain."""
    tds = [plan["tds"][i] for i in range(plan["n_tds"])]
    counters = [0] * max(1, plan["n_events"])
    nxt, holding, done = 0, [None] * workers, 0
    for _ in range(10 * len(tds) + 10):
        progressed = False
        for w in range(workers):
            if holding[w] is None and nxt < len(tds):
                holding[w] = tds[nxt]; nxt += 1; progressed = True
            td = holding[w]
            if td is not None and (td.dependent_event == NONE or counters[td.dependent_event] >= td.dependent_threshold):
                if td.trigger_event != NONE:
                    counters[td.trigger_event] += 1
                holding[w] = None; done += 1; progressed = True
        if done == len(tds):
            return counters
        assert progressed, "deadlock"
    raise AssertionError("did not finish")


def test_split_propagation_labels_and_task_counts():
    tensors, ops = _pair(M=100, rows_a=8, rows_b=8)
    plan = B.moe_taskflow_compile(tensors, ops, lag_rows=32)
    assert plan["op_task_num"] == [13, 13]                       # ceil(100 / 8)
    assert plan["tensor_split_dim"] == [-1, 0, -1, 0]            # labels sit on produced tensors only
    assert plan["tensor_split_num"] == [1, 13, 1, 13]
    assert plan["n_tds"] == 26 and plan["n_events"] == 13
    tds = [plan["tds"][i] for i in range(plan["n_tds"])]
    sw = [t for t in tds if t.task_type == SW]
    ad = [t for t in tds if t.task_type == ADD]
    assert sorted(t.task_index for t in sw) == list(range(13)) == sorted(t.task_index for t in ad)
    for t in sw:
        assert t.dependent_event == NONE and t.trigger_event == t.task_index
        assert (t.inputs[0].slot, t.inputs[0].cols, t.outputs[0].slot, t.outputs[0].cols) == (0, 128, 1, 64)
        assert t.outputs[0].row_offset == 8 * t.task_index and t.outputs[0].rows == (4 if t.task_index == 12 else 8)
        assert t.task_split_num == 13 and t.task_split_value == 8 and t.tiling_data_position == 0
    for t in ad:
        assert t.dependent_event == t.task_index and t.dependent_threshold == 1 and t.trigger_event == NONE
        assert [t.inputs[i].slot for i in range(2)] == [1, 2] and t.outputs[0].slot == 3


def test_unmet_split_requirement_falls_back_to_one_unsplit_task():
    # Add asks for its first input to be split along dimension 1; SwiGLU labels it along 0 -> one task, whole tensor
    tensors, ops = _pair(M=100, add_split=((0, 1),))
    plan = B.moe_taskflow_compile(tensors, ops, lag_rows=0)
    assert plan["op_task_num"] == [13, 1]
    assert plan["tensor_split_dim"][3] == -1 and plan["tensor_split_num"][3] == 1
    tds = [plan["tds"][i] for i in range(plan["n_tds"])]
    add = [t for t in tds if t.task_type == ADD]
    assert len(add) == 1 and add[0].outputs[0].rows == 100 and add[0].dependent_threshold == 13   # waits for every tile
    assert tds[-1].task_type == ADD                                # and is ordered behind all of them
    assert plan["n_events"] == 1
    # an unsplit producer writes no label (n = 1), so a consumer that asks for one falls back too -- Algorithm 1's rule
    tensors, ops = _pair(M=64, rows_a=64, rows_b=8)
    plan = B.moe_taskflow_compile(tensors, ops, lag_rows=0)
    assert plan["op_task_num"] == [1, 1] and plan["tensor_split_dim"][1] == -1
    # a consumer that is a partition origin of its own splits anyway: its tiles all wait on the producer's one event
    tensors = [(64, 128), (64, 64), (64, 64), (64, 64)]
    ops = [B.tf_operator(SW, [0], [1], 64, split_inputs=None), B.tf_operator(ADD, [1, 2], [3], 8, split_inputs=None)]
    plan = B.moe_taskflow_compile(tensors, ops, lag_rows=0)
    assert plan["op_task_num"] == [1, 8] and plan["n_events"] == 1
    tds = [plan["tds"][i] for i in range(plan["n_tds"])]
    assert tds[0].task_type == SW and all(t.dependent_event == 0 and t.dependent_threshold == 1 for t in tds[1:])


def test_granularities_that_nest_share_events_with_thresholds():
    tensors, ops = _pair(M=96, rows_a=8, rows_b=32)                # four producers per consumer tile
    plan = B.moe_taskflow_compile(tensors, ops, lag_rows=32)
    tds = [plan["tds"][i] for i in range(plan["n_tds"])]
    assert plan["op_task_num"] == [12, 3] and plan["n_events"] == 3
    assert all(t.dependent_threshold == 4 for t in tds if t.task_type == ADD)
    assert all(t.trigger_event == t.task_index // 4 for t in tds if t.task_type == SW)
    tensors, ops = _pair(M=96, rows_a=32, rows_b=8)                # four consumers per producer tile
    plan = B.moe_taskflow_compile(tensors, ops, lag_rows=32)
    tds = [plan["tds"][i] for i in range(plan["n_tds"])]
    assert all(t.dependent_threshold == 1 and t.dependent_event == t.task_index // 4 for t in tds if t.task_type == ADD)
    with pytest.raises(B.MoeError):
        B.moe_taskflow_compile(*_pair(M=96, rows_a=8, rows_b=12), lag_rows=0)   # 12 is not a multiple of 8


@pytest.mark.parametrize("lag", [0, 8, 64, 1000])
@pytest.mark.parametrize("workers", [1, 3, 592])
def test_queue_order_is_topological_and_drains_for_any_worker_count(lag, workers):
    tensors, ops = _pair(M=500, rows_a=8, rows_b=16)
    plan = B.moe_taskflow_compile(tensors, ops, lag_rows=lag)
    tds = [plan["tds"][i] for i in range(plan["n_tds"])]
    raised = {}
    for t in tds:                                                  # every producer of an event sits before its waiters
        if t.dependent_event != NONE:
            assert raised.get(t.dependent_event, 0) == t.dependent_threshold
        if t.trigger_event != NONE:
            raised[t.trigger_event] = raised.get(t.trigger_event, 0) + 1
    counters = _simulate(plan, workers)
    for t in tds:
        if t.dependent_event != NONE:
            assert counters[t.dependent_event] == t.dependent_threshold
    if lag == 64:                                                  # a consumer runs `lag` rows behind its producers
        pos = {(t.task_type, t.task_index): i for i, t in enumerate(tds)}
        assert pos[(ADD, 0)] > pos[(SW, 7)] and pos[(ADD, 0)] < pos[(SW, 12)]


def test_three_operator_chain_and_a_diamond():
    M, C = 64, 32
    # x -> SwiGLU -> s ; s + r -> z1 ; z1 + s -> z2   (s has two consumers; z1 and s are consumed together)
    tensors = [(M, 2 * C), (M, C), (M, C), (M, C), (M, C)]
    ops = [B.tf_operator(SW, [0], [1], 8, split_inputs=None),
           B.tf_operator(ADD, [1, 2], [3], 8, split_inputs=[(0, 0)]),
           B.tf_operator(ADD, [3, 1], [4], 8, split_inputs=[(0, 0), (1, 0)])]
    plan = B.moe_taskflow_compile(tensors, ops, lag_rows=16)
    assert plan["op_task_num"] == [8, 8, 8]
    assert plan["n_tds"] == 24
    _simulate(plan, 5)


def test_rejects_malformed_graphs():
    tensors, ops = _pair()
    with pytest.raises(B.MoeError):
        B.moe_taskflow_compile(tensors, [ops[0], ops[0]], 0)                 # two writers of one tensor
    with pytest.raises(B.MoeError):
        B.moe_taskflow_compile([(100, 64), (100, 64), (100, 64), (100, 64)], ops, 0)   # SwiGLU needs 2C input columns
    cyc = [B.tf_operator(ADD, [1, 2], [3], 8, split_inputs=None), B.tf_operator(ADD, [3, 2], [1], 8, split_inputs=None)]
    with pytest.raises(B.MoeError):
        B.moe_taskflow_compile([(8, 16)] * 4, cyc, 0)                         # a cycle
    with pytest.raises(B.MoeError):
        B.moe_taskflow_compile(tensors, ops, 0, td_cap=3)                     # descriptor array too small
