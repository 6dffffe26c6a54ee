"""The five benchmark / parity workloads of the HMAR attention path.

Shapes follow the paper's attention micro-benchmark (App. B.4: batch 16, head dim 64,
number of heads equal to the model depth) and its K = 10 resolution scales (Sec. 4.3).
The side-length schedules are those of the VAR tokenizer family the paper builds on; the
paper itself prints only K = 10 and the 1..16 range for 256x256 images.
"""
from dataclasses import dataclass
from typing import Tuple

SIDES_TINY = (1, 2, 3, 4)
SIDES_256 = (1, 2, 3, 4, 5, 6, 8, 10, 13, 16)
SIDES_512 = (1, 2, 3, 4, 6, 9, 13, 18, 24, 32)
# 1024x1024: the paper benchmarks this resolution (App. B.4) but prints no schedule for it; this one is
# synthetic (the 512 schedule's growth continued to a 64 x 64 last scale, 14 scales).
SIDES_1024 = (1, 2, 3, 4, 5, 7, 9, 12, 16, 21, 27, 36, 48, 64)

BASE_SEED = 20250604 * 10


@dataclass(frozen=True)
class Workload:
    name: str
    index: int                 # position in the config list (1-based)
    B: int
    H: int
    D: int
    side_lens: Tuple[int, ...]
    softmax_scale: float
    passes: Tuple[str, ...]    # subset of ("fwd", "bwd", "scale_step")
    sub_steps: int = 1         # inference: masked refinement sub-steps per scale

    @property
    def seed(self) -> int:
        return BASE_SEED + self.index

    @property
    def L(self) -> int:
        return sum(s * s for s in self.side_lens)


CONFIGS = {
    "tiny": Workload("tiny", 1, 1, 2, 64, SIDES_TINY, 0.125, ("fwd", "bwd")),
    "256_d16_fwd": Workload("256_d16_fwd", 2, 8, 16, 64, SIDES_256, 0.125, ("fwd",)),
    "256_d30_train": Workload("256_d30_train", 3, 32, 30, 64, SIDES_256, 0.125, ("fwd", "bwd")),
    "512_d24_train": Workload("512_d24_train", 4, 16, 24, 64, SIDES_512, 0.125, ("fwd", "bwd")),
    "512_d24_infer": Workload("512_d24_infer", 5, 64, 24, 64, SIDES_512, 0.125, ("scale_step",), 4),
    "1024_d24_train": Workload("1024_d24_train", 6, 16, 24, 64, SIDES_1024, 0.125, ("fwd", "bwd")),
}


def get_config(name: str) -> Workload:
    return CONFIGS[name]
