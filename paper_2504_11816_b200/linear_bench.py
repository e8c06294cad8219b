"""Times the decode linear layers (``isv_linear_forward``) on the GPU at hand.

    python -m paper_2504_11816_b200.linear_bench [--batch 32] [--model llama7b|opt2.7b]

For each projection of one transformer layer (fused QKV, output, MLP up, MLP down) the weight
matrix is streamed once per call; the figure of merit is weight bytes / time against the HBM
peak.  Several distinct weight buffers are cycled so that no call finds its weights in L2.
Prints one JSON object.  Needs a CUDA device.
"""
from __future__ import annotations

import argparse
import json
import os

MODELS = {
    # name: (h1, h2, gated MLP)
    "llama7b": (4096, 11008, True),
    "opt2.7b": (2560, 10240, False),
}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--batch", type=int, default=32)
    ap.add_argument("--model", default="llama7b", choices=sorted(MODELS))
    ap.add_argument("--iters", type=int, default=40)
    ap.add_argument("--eager", action="store_true", help="time the plain call loop instead of a captured graph")
    args = ap.parse_args()
    import torch
    from . import binding as B
    assert torch.cuda.is_available(), "needs a CUDA device"
    h1, h2, gated = MODELS[args.model]
    shapes = [("qkv", 3 * h1, h1), ("out", h1, h1), ("mlp_up", (2 if gated else 1) * h2, h1), ("mlp_down", h1, h2)]
    peak = 6650.0
    pk = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "MEASURED_PEAKS.json")
    if os.path.exists(pk):
        peak = float(json.load(open(pk))["hbm_gbs"])
    stream = torch.cuda.Stream()
    M = args.batch
    rows = []
    total_s = 0.0
    for name, N, K in shapes:
        wbytes = N * K * 2
        copies = max(2, int((512 << 20) // wbytes) + 1)          # > L2 in total
        g = torch.Generator(device="cuda")
        g.manual_seed(N * 31 + K)
        ws = [(torch.randn((N, K), generator=g, device="cuda", dtype=torch.float32) / K ** 0.5).half()
              for _ in range(copies)]
        x = torch.randn((M, K), generator=g, device="cuda", dtype=torch.float32).half()
        y = torch.zeros((M, N), device="cuda", dtype=torch.float16)
        torch.cuda.synchronize()
        hs = [B.isv_linear_create(w, N, K, B.ISV_F16, max(M, 16), stream.cuda_stream) for w in ws]
        try:
            for h in hs:
                B.isv_linear_forward(h, x, y, None, M)
            assert B.isv_linear_status(hs[0]) == 0
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            # The calls are captured into a CUDA graph and the graph is timed: a projection of a few
            # microseconds is otherwise bound by the host's launch rate (Python call + tensor-map encoding
            # + launch), which says nothing about the kernel.  --eager times the plain call loop instead.
            graph = None
            if not args.eager:
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph, stream=stream):
                    for i in range(args.iters):
                        B.isv_linear_forward(hs[i % copies], x, y, None, M)
                graph.replay()                                  # warm-up replay
                stream.synchronize()
                torch.cuda.synchronize()
            with torch.cuda.stream(stream):
                e0.record(stream)
                if graph is not None:
                    graph.replay()
                else:
                    for i in range(args.iters):
                        B.isv_linear_forward(hs[i % copies], x, y, None, M)
                e1.record(stream)
            stream.synchronize()
            torch.cuda.synchronize()
            t = e0.elapsed_time(e1) * 1e-3 / args.iters
            # agreement with a library GEMM on the last call's output
            ref = torch.nn.functional.linear(x.float(), ws[(args.iters - 1) % copies].float())
            err = float((y.float() - ref).abs().max())
        finally:
            for h in hs:
                B.isv_linear_free(h)
        rows.append({"layer": name, "N": N, "K": K, "us": t * 1e6, "weight_GBps": wbytes / t / 1e9,
                     "frac_of_hbm_peak": wbytes / t / 1e9 / peak, "TFLOPs": 2.0 * M * N * K / t / 1e12,
                     "max_abs_diff_vs_fp32_gemm": err})
        total_s += t
        del ws
        torch.cuda.empty_cache()
    flops = 2.0 * M * sum(N * K for _, N, K in shapes)
    print(json.dumps({"device": torch.cuda.get_device_name(0), "model": args.model, "batch": M, "hbm_peak_GBps": peak,
                      "timed": "plain call loop" if args.eager else "CUDA graph of the calls",
                      "rows": rows, "linear_s_per_layer": total_s, "linear_flops_per_layer": flops,
                      "weights_GBps_overall": sum(r["N"] * r["K"] * 2 for r in rows) / total_s / 1e9}))


if __name__ == "__main__":
    main()
