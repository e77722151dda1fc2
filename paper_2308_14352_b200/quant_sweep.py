"""Quantisation variants side by side (paper Section 3.2: channel-wise linear quantisation; the
text leaves the scale granularity and the exact code range open).  For one seeded expert FFN the
same fp32 weights are packed by the library at every width, with one scale per output channel or
per group of 64 / 128 inputs, and with the symmetric or the full code range; the layer then runs
through the library's forward call and its output is compared with the output of the unquantised
weights (a plain fp64 matmul on the device, the reference of this tool only).

    python -m paper_2308_14352_b200.quant_sweep [--d-model 1024 --d-ff 4096 --tokens 32 --act relu]

Prints one markdown table: bits, scale layout, range reading, stored bytes per weight, and the
relative output error  ||y_q - y_fp|| / ||y_fp||.
"""
from __future__ import annotations

import argparse

import numpy as np
import torch

from . import binding as B, inputs, layer


def reference_output(x: torch.Tensor, W, act: str) -> torch.Tensor:
    """The expert FFN on unquantised weights in fp64; the hidden vector is rounded to bf16 as the
    library's is, so that the difference left is the quantisation's."""
    xd = x.double()
    if act == "relu":
        h = torch.relu(xd @ W[0].double().T)
    else:
        a = xd @ W[0].double().T
        h = a / (1.0 + torch.exp(-a)) * (xd @ W[1].double().T)
    h = h.float().bfloat16().double()
    return h @ W[-1].double().T


def run(d_model: int, d_ff: int, tokens: int, act: str, seed: int, outliers: float):
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    gen = torch.Generator(device=dev)
    gen.manual_seed(seed)
    n_mat = 2 if act == "relu" else 3
    W = []
    for m in range(n_mat):
        N, K = (d_ff, d_model) if m < n_mat - 1 else (d_model, d_ff)
        w = torch.randn(N, K, generator=gen, device=dev) * 0.02
        if outliers > 0:  # a few weights far out, as trained matrices have: they set max-abs and so the scale
            mask = torch.rand(N, K, generator=gen, device=dev) < outliers
            w = torch.where(mask, w * 8.0, w)
        W.append(w.contiguous())
    x = torch.randn(tokens, d_model, generator=gen, device=dev).bfloat16()
    y_ref = reference_output(x, W, act)
    ids = torch.zeros(tokens, 1, dtype=torch.int32, device=dev)
    gates = torch.ones(tokens, 1, dtype=torch.float32, device=dev)
    rows = []
    for bits in (8, 4, 2):
        for group, sdt in ((0, "f32"), (128, "f16"), (64, "f16")):
            for full in (False, True):
                shape = inputs.LayerShape(d_model, d_ff, 1, 1, act, "softmax", group, sdt, "bf16")
                with layer.MoELayer(shape, [bits], max_tokens=tokens) as moe:
                    for m in range(n_mat):
                        moe.pack_matrix(0, m, W[m], full_range=full)
                    y = torch.empty(tokens, d_model, dtype=torch.float32, device=dev)
                    B.emoe_moe_forward_routed(moe.ctx, moe.desc, x.data_ptr(), tokens, ids.data_ptr(), gates.data_ptr(),
                                              moe.table, y.data_ptr(), None, 0)
                    torch.cuda.synchronize(dev)
                    st = B.emoe_device_status(moe.ctx)
                    if st != B.OK:
                        raise B.EmoeError(st, "emoe_moe_forward_routed (device check)")
                err = float((y.double() - y_ref).norm() / y_ref.norm())
                G = group or d_model
                bytes_per_weight = bits / 8 + (2 if sdt == "f16" else 4) / G
                rows.append((bits, "per channel (fp32)" if group == 0 else f"group {group} (fp16)",
                             "full" if full else "symmetric", bytes_per_weight, err))
    return rows


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--d-model", type=int, default=1024)
    ap.add_argument("--d-ff", type=int, default=4096)
    ap.add_argument("--tokens", type=int, default=32)
    ap.add_argument("--act", choices=("relu", "swiglu"), default="relu")
    ap.add_argument("--seed", type=int, default=7)
    ap.add_argument("--outliers", type=float, default=0.001, help="fraction of weights scaled by 8")
    a = ap.parse_args()
    rows = run(a.d_model, a.d_ff, a.tokens, a.act, a.seed, a.outliers)
    print(f"expert FFN {a.d_model} x {a.d_ff} ({a.act}), {a.tokens} tokens, N(0, 0.02) weights, "
          f"{a.outliers:g} of them x 8; error = ||y_q - y_fp|| / ||y_fp||")
    print("| bits | scales | code range | bytes per weight | output error |")
    print("|---|---|---|---|---|")
    for bits, lay, rng, bpw, err in rows:
        print(f"| {bits} | {lay} | {rng} | {bpw:.4f} | {err:.4f} |")


if __name__ == "__main__":
    main()
