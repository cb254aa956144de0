"""Device-side timing helpers shared by bench.py and the sweep."""
from __future__ import annotations

import torch


def kernel_ms_back_to_back(launch, launches: int) -> float:
    """Mean device time of one launch when the kernel runs back to back: `launches` launches replayed from CUDA
    graphs of ten (so the host's launch cost cannot stretch the figure), one event pair around all of them."""
    per_graph = 10
    launch()
    g = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        with torch.cuda.graph(g, stream=side):
            for _ in range(per_graph):
                launch()
    torch.cuda.current_stream().wait_stream(side)
    replays = max(1, launches // per_graph)
    g.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(replays):
        g.replay()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / (replays * per_graph)
