"""Shared helpers of the GPU parity tests (CUDA path through the C ABI vs the CPU oracle)."""
import torch

from oracle.specvla import SpecVLAOracle, Tree
from synth_inputs import configs as C, data

MARGIN = 5e-2        # tokens must agree wherever the oracle's top-2 margin exceeds this
LOGIT_TOL = 2e-2     # max-abs logit difference, bf16 path vs float64 oracle


def to_cuda(weights):
    return {k: v.cuda().contiguous() for k, v in weights.items()}


def make_gpu(desc, weights_cuda, **kw):
    from paper_2507_22424_b200.binding import SpecVLA
    return SpecVLA(desc, weights_cuda, **kw)


def tree_dict(t: Tree):
    return dict(tokens=list(t.tokens), parent=list(t.parent), depth=list(t.depth))


def margins(logits, desc, action_only):
    """Top-1 minus top-2 per row of an oracle logits matrix."""
    if action_only:
        logits = logits[:, desc.action_base:desc.action_base + desc.n_bins]
    top = torch.topk(logits, 2, dim=1).values
    return (top[:, 0] - top[:, 1])


def compare_tokens(gpu_tokens, oracle_tokens, margin_list, log, where):
    """Bit-exact wherever the margin is large; every low-margin position is logged."""
    for i, (a, b, mg) in enumerate(zip(gpu_tokens, oracle_tokens, margin_list)):
        if mg <= MARGIN:
            log.append(f"{where}[{i}]: margin {mg:.4f} <= {MARGIN} (gpu {a}, oracle {b})")
        else:
            assert a == b, f"{where}[{i}]: gpu {a} != oracle {b} at margin {mg:.4f}"
