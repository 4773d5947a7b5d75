"""Every launch entry only enqueues work on the caller's stream, so a sequence of calls can be captured into a
CUDA graph and replayed: the replay must give the same outputs as the direct calls, and match the oracle.
"""
import numpy as np
import pytest

from helpers import FFMA_TOL, TF32_TOL, assert_parity
from workloads import uniform

pytestmark = pytest.mark.gpu


def test_calls_captured_in_a_cuda_graph_replay_correctly(oracle):
    import torch
    import paper_1705_10591_b200 as lib

    dev = torch.device("cuda:0")
    # (entry, N, C, H, W, K, R, S, algo)
    cases = [("single", 1, 1, 40, 132, 6, 3, 3, lib.ALGO_FFMA),
             ("general", 2, 48, 18, 20, 72, 3, 3, lib.ALGO_TF32),      # tensor cores, filters re-ordered inside the graph
             ("general", 1, 160, 9, 11, 40, 5, 5, lib.ALGO_TF32),      # stacked taps, split contraction (zero-fill node)
             ("general", 2, 20, 15, 16, 70, 3, 3, lib.ALGO_FFMA)]
    bufs = []
    for i, (entry, N, C, H, W, K, R, S, algo) in enumerate(cases):
        x, w = uniform((N, C, H, W), 481 + 2 * i), uniform((K, C, R, S), 482 + 2 * i)
        xd, wd = torch.from_numpy(x).to(dev), torch.from_numpy(w).to(dev)
        yd = torch.full((N, K, H - R + 1, W - S + 1), float("nan"), device=dev)
        nbytes = 0 if entry == "single" else lib.conv2d_fwd_workspace_size(N, C, H, W, K, R, S, algo)
        ws = torch.zeros(max(nbytes, 16), dtype=torch.uint8, device=dev)
        bufs.append((x, w, xd, wd, yd, ws, nbytes))

    def enqueue(stream):
        for (entry, N, C, H, W, K, R, S, algo), (_, _, xd, wd, yd, ws, nbytes) in zip(cases, bufs):
            if entry == "single":
                lib.conv2d_fwd_single_channel(xd.data_ptr(), wd.data_ptr(), yd.data_ptr(), N, H, W, K, R, S, 0, 0, 0, stream)
            else:
                lib.conv2d_fwd_general(xd.data_ptr(), wd.data_ptr(), yd.data_ptr(), N, C, H, W, K, R, S, algo,
                                       ws.data_ptr() if nbytes else 0, nbytes, 0, stream)

    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        enqueue(side.cuda_stream)                       # warm-up outside the capture (one-time kernel attributes)
    side.synchronize()
    direct = [b[4].clone() for b in bufs]
    for b in bufs:
        b[4].fill_(float("nan"))

    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        enqueue(torch.cuda.current_stream().cuda_stream)
    for b in bufs:                                       # capturing must not have run anything
        assert torch.isnan(b[4]).all().item()
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()

    for (entry, N, C, H, W, K, R, S, algo), (x, w, _, _, yd, ws, nbytes), y_direct in zip(cases, bufs, direct):
        got = yd.cpu().numpy()
        y_ref, yabs = oracle.conv2d_oracle(x, w)
        tol = TF32_TOL if algo == lib.ALGO_TF32 else FFMA_TOL
        assert_parity(got, y_ref, yabs, tol, f"graph replay {entry} {(N, C, H, W, K, R, S)}")
        np.testing.assert_array_equal(got, y_direct.cpu().numpy())
        if nbytes:
            lib.conv2d_get_status(ws.data_ptr(), torch.cuda.current_stream().cuda_stream)
