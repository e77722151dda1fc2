"""Shared helpers of the GPU parity tests: oracle-side packing of a layer and the metrics."""
import numpy as np

import oracle
from paper_2308_14352_b200 import inputs


def oracle_pack_layer(W, shape, bits, full_range=False):
    packed, scales = [], []
    for e in range(shape.n_experts):
        ps = [oracle.pack_expert(W[e][m], bits[e], shape.group, shape.scale_dtype, full_range)
              for m in range(shape.n_matrices)]
        packed.append([p for p, _ in ps])
        scales.append([s for _, s in ps])
    return packed, scales


def rel_to_max(y, ref):
    """max |y - ref| / max |ref|: the output metric of the parity bar."""
    return float(np.abs(y.astype(np.float64) - ref.astype(np.float64)).max() / np.abs(ref).max())


def output_tolerance(act_dtype):
    """2e-3 with bf16 activations, 1e-5 with fp32 activations."""
    return 2e-3 if act_dtype == "bf16" else 1e-5


def check_ids(ids_gpu, logits_ref, k, margin=1e-4):
    """Expert ids must equal the oracle's wherever every decisive logit gap exceeds `margin`;
    elsewhere any pick whose logit is within `margin` of the oracle's pick at that rank is valid.
    Returns the number of rows where the comparison was strict."""
    order = np.argsort(-logits_ref, axis=1, kind="stable")
    strict = 0
    for t in range(ids_gpu.shape[0]):
        z = logits_ref[t]
        srt = z[order[t]]
        gaps = srt[:k] - srt[1:k + 1] if z.size > k else srt[:k - 1] - srt[1:k]
        if gaps.size == 0 or gaps.min() > margin:
            assert np.array_equal(ids_gpu[t], order[t, :k]), (t, ids_gpu[t], order[t, :k])
            strict += 1
        else:
            for j in range(k):
                assert abs(z[ids_gpu[t, j]] - srt[j]) <= margin
            assert len(set(ids_gpu[t].tolist())) == k
    return strict
