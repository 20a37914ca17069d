"""Runs shape lists through the guarded build of the library (RCP_W2A4_LIB points at it) and checks that no
guard fired (status word 0) and that the results are the production build's, which the parent test passes in a
file. Started as a child process by tests/test_gpu_checked_build.py: one process loads one build."""
import sys

import numpy as np
import torch

import paper_2502_15779_b200 as rcp
from gen import synth

DEV = "cuda:0"


def run(cases):
    out = {}
    for i, (N, K, B, M, variant, grouped) in enumerate(cases):
        seed = 100 + i
        if grouped:
            codes, lut = synth.make_layer_grouped(N, K, 128, B, "uniform", seed, device=DEV)
        else:
            codes, lut = synth.make_layer(N, K, B, "uniform", seed, device=DEV)
        x = synth.make_activations(M, K, seed, device=DEV)
        words = rcp.rcp_pack_weights(codes)
        xq, scale = rcp.rcp_quantize_act(x, B, 1.0)
        ws = rcp.make_workspace(M, N, K, DEV)
        if variant == "linear":
            y = rcp.rcp_linear_w2a4(x, B, 1.0, words, lut, group=128 if grouped else 0, xq=xq, scale=scale, workspace=ws)
        elif variant == "w2a16":
            y = rcp.rcp_gemv_w2a16(words, lut, x, workspace=ws)
        elif grouped:
            y = rcp.rcp_gemv_w2a4_grouped(words, lut, xq, scale, group=128, workspace=ws, variant=variant)
        else:
            y = rcp.rcp_gemv_w2a4(words, lut, xq, scale, workspace=ws, variant=variant)
        torch.cuda.synchronize()
        out[f"status{i}"] = ws.cpu().numpy()[:1].copy()
        out[f"y{i}"] = y.cpu().view(torch.int16).numpy().copy()
    return out


if __name__ == "__main__":
    from test_gpu_checked_build import CASES
    np.savez(sys.argv[1], **run(CASES))
