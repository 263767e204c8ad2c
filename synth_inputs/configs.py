"""Shapes of the synthetic workloads (model, prefix, draft tree) and their seeds.

Only sizes, seeds and stream numbers live here. The workloads stand in for the paper's
LIBERO episodes (Section 5.1): 256 visual patch embeddings followed by a short text
prompt, seven action tokens per chunk, 256 action bins.
"""
from __future__ import annotations

from dataclasses import dataclass, field, asdict


@dataclass(frozen=True)
class ModelDesc:
    n_layers: int
    d_model: int
    n_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    action_base: int          # id of action bin 0
    n_bins: int = 256
    rms_eps: float = 1e-6
    rope_theta: float = 1e4

    def as_dict(self):
        return asdict(self)


@dataclass(frozen=True)
class TreeShape:
    """Static-size draft tree: level l has expand[l] * branch[l] nodes.

    expand[l] parents of level l-1 (the root for l = 0) are expanded, each into
    branch[l] children.
    """
    branch: tuple
    expand: tuple
    keep: int = 0             # > 0: after the last level only the `keep` best nodes are verified

    @property
    def depth(self):
        return len(self.branch)

    @property
    def level_sizes(self):
        return tuple(b * e for b, e in zip(self.branch, self.expand))

    @property
    def n_nodes(self):
        return sum(self.level_sizes)


@dataclass(frozen=True)
class Workload:
    name: str
    model: ModelDesc
    seed: int
    n_visual: int
    visual_scale: float
    n_text: tuple             # (lo, hi) inclusive range of text-token counts
    tree: TreeShape
    n_tokens: int = 7
    action_only: int = 1
    extra: dict = field(default_factory=dict)


TINY = ModelDesc(n_layers=2, d_model=256, n_heads=4, head_dim=64, d_ffn=688,
                 vocab=1024, action_base=768)
OPENVLA_7B = ModelDesc(n_layers=32, d_model=4096, n_heads=32, head_dim=128, d_ffn=11008,
                       vocab=32064, action_base=31744)

TREE_C0 = TreeShape(branch=(2, 2, 2), expand=(1, 2, 4))                  # 2+4+8 = 14 nodes
TREE_26 = TreeShape(branch=(4, 2, 2, 1, 1), expand=(1, 4, 3, 4, 4))      # 4+8+6+4+4 = 26 nodes

C0 = Workload("C0-tiny", TINY, seed=0, n_visual=64, visual_scale=1.0, n_text=(0, 0),
              tree=TREE_C0)
C1 = Workload("C1-openvla7b-bs1", OPENVLA_7B, seed=1, n_visual=256, visual_scale=0.5,
              n_text=(34, 34), tree=TREE_26)
C2 = Workload("C2-relaxed-sweep", OPENVLA_7B, seed=1, n_visual=256, visual_scale=0.5,
              n_text=(34, 34), tree=TREE_26, extra={"r": (0, 1, 2, 4, 8, 16)})
C3 = Workload("C3-verify-roofline", OPENVLA_7B, seed=1, n_visual=256, visual_scale=0.5,
              n_text=(34, 41), tree=TREE_26,
              extra={"rows": (1, 8, 26, 60, 128), "tree_seed": 2, "max_depth": 8})
C4 = Workload("C4-batched-16", OPENVLA_7B, seed=1, n_visual=256, visual_scale=0.5,
              n_text=(20, 60), tree=TREE_26, extra={"episodes": 16, "prefix_seed": 3, "r": 4})

# Stream numbers of the counter-based generator (one per tensor).
STREAM_EMBED = 1
STREAM_LM_HEAD = 2
STREAM_DRAFT_FC = 50
STREAM_DRAFT_LAYER = 60          # +0 q, +1 k, +2 v, +3 o, +4 gate, +5 up, +6 down
STREAM_LAYER0 = 100              # + 10 * layer + (0 q, 1 k, 2 v, 3 o, 4 gate, 5 up, 6 down)
STREAM_VISUAL = 1000             # + episode
STREAM_TEXT_IDS = 1100           # + episode
STREAM_TEXT_LEN = 1200
STREAM_TREE_PARENT = 2000
STREAM_TREE_TOKEN = 2001
STREAM_PLANT = 3000              # + call counter
