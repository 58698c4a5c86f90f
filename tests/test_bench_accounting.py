"""Host-side checks of the byte and flop accounting that bench.py divides device times into."""
import importlib.util
import os

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _bench():
    spec = importlib.util.spec_from_file_location("bench_module", os.path.join(ROOT, "bench.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


CFG = dict(dims=[3072, 2048, 2048, 2048, 10], P=32, K=16, B=64)


def test_plain_schedule_moves_fourteen_bytes_per_weight_and_step():
    b = _bench()
    per = b.algorithmic_bytes(CFG, tensor_path=False)
    nW = [3072 * 2048, 2048 * 2048, 2048 * 2048, 2048 * 10]
    P, K, rows = 32, 16, 32 * 64
    assert per["wgrad_sgd_gemm"]["bytes"] == K * (P * 10 * sum(nW) + 2 * rows * sum(CFG["dims"]))
    assert per["fwd_gemm"]["flops"] == per["wgrad_sgd_gemm"]["flops"] == K * 2 * rows * sum(nW)
    weights = (per["fwd_gemm"]["bytes"] + per["dgrad_gemm"]["bytes"] + per["wgrad_sgd_gemm"]["bytes"])
    # 2 (forward) + 2 (dgrad, not for layer 1) + 10 bytes per weight, plus activations
    assert weights > K * P * (14 * sum(nW) - 2 * nW[0])
    assert weights < 1.06 * K * P * 14 * sum(nW)


def test_riding_and_dense_forward_only_move_work_between_classes_and_remove_bytes():
    b = _bench()
    plain = b.algorithmic_bytes(CFG, tensor_path=True)
    ride = b.algorithmic_bytes(CFG, tensor_path=True, fwd_run_tiles=(48, 32, 32),
                               dense_layers=(1, 2, 3), fwd_whole_rows=(444, 444, 444))
    nW = [3072 * 2048, 2048 * 2048, 2048 * 2048]
    P, K, B = 32, 16, 64
    # flops are conserved; the hidden layers' forward flops of steps 2..K are in the other class
    total = lambda d: sum(v["flops"] for v in d.values())
    assert total(plain) == total(ride)
    moved = (K - 1) * 2 * P * B * sum(nW)
    assert ride["wgrad_sgd_gemm"]["flops"] - plain["wgrad_sgd_gemm"]["flops"] == moved
    # bytes: per riding step 2 B per hidden weight less read by forward kernels, 2 B per layer-1
    # weight less written; the first step reads the hidden layers' weights once, not P times;
    # the partial sums of the 68 cut rows (two runs each) come on top, written and read
    saved = (K - 1) * 2 * P * (sum(nW) + nW[0]) + 2 * (P - 1) * sum(nW)
    partial = (K - 1) * 3 * 2 * (68 * 2 * B * 128 * 4)
    tot_b = lambda d: sum(v["bytes"] for v in d.values())
    assert tot_b(plain) - tot_b(ride) == saved - partial
    # whole rows only: no partial sums at all
    whole = b.algorithmic_bytes(CFG, tensor_path=True, fwd_run_tiles=(96, 64, 64),
                                dense_layers=(1, 2, 3), fwd_whole_rows=(512, 512, 512))
    assert tot_b(plain) - tot_b(whole) == saved
