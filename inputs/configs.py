"""The five workloads: network shape, precision, batch size and the seeds of their inputs.

Pure data.  `arch` fields use the same integer codes as the library's arch struct:
policy_head 0 = 73 move planes (4672 logits), 1 = flat 1858-move list;
value_head 0 = scalar tanh, 1 = win/draw/loss softmax;
precision 0 = fp32, 1 = bf16, 2 = FP8-e4m3 tower (heads bf16), 3 = int8 tower (heads bf16),
4 = FP8-e4m3 tower with every operand as a pair of e4m3 numbers, 5 = pairs for the activations only.
"""
from dataclasses import dataclass, field
from typing import Tuple

POLICY_SIZE = {0: 73 * 64, 1: 1858}
MASK_WORDS = {0: 73, 1: 30}
VALUE_SIZE = {0: 1, 1: 3}
HEAD_CHANNELS = 32      # 1x1-conv width of the flat policy head and of the value head
VALUE_HIDDEN = 128


@dataclass(frozen=True)
class Config:
    name: str
    in_planes: int
    blocks: int
    channels: int
    policy_head: int
    value_head: int
    precision: int
    batch: int
    plies_even: Tuple[int, int]
    plies_odd: Tuple[int, int]
    position_seed: int
    weight_seed: int
    weights_like: str = ""       # name of the config whose weights (and head scales) this one reuses
    branch_scale: float = 1.0    # factor folded into every block's second scale and bias (1/sqrt(blocks) in c4b)
    sweep: Tuple[int, ...] = field(default_factory=tuple)

    @property
    def policy_size(self) -> int:
        return POLICY_SIZE[self.policy_head]

    @property
    def mask_words(self) -> int:
        return MASK_WORDS[self.policy_head]

    @property
    def value_size(self) -> int:
        return VALUE_SIZE[self.value_head]

    @property
    def weights_name(self) -> str:
        return self.weights_like or self.name


CONFIGS = {
    "c1": Config("c1", 19, 6, 64, 0, 0, 0, 64, (0, 80), (0, 80), 20260938, 9370001),
    "c2": Config("c2", 19, 20, 128, 0, 0, 1, 256, (0, 80), (0, 80), 20260939, 9370002),
    "c3": Config("c3", 19, 20, 128, 1, 1, 1, 1024, (0, 40), (40, 160), 20260940, 9370003),
    "c4": Config("c4", 19, 20, 128, 0, 0, 2, 4096, (0, 80), (0, 80), 20260941, 9370002, weights_like="c2"),
    # c4 with the residual branches scaled by 1/sqrt(depth), the paper's quantisation-friendly block
    # (Sec. 4.3.6), folded into the second convolution's scale and bias as the paper does at export
    "c4b": Config("c4b", 19, 20, 128, 0, 0, 2, 4096, (0, 80), (0, 80), 20260941, 9370002, branch_scale=20 ** -0.5),
    # the same network with the tower in int8 (unsigned 8-bit activations, signed 8-bit weights), the
    # precision the paper deploys (Sec. 4.3.6); precision code 3
    "c4i": Config("c4i", 19, 20, 128, 0, 0, 3, 4096, (0, 80), (0, 80), 20260941, 9370002, weights_like="c4b",
                  branch_scale=20 ** -0.5),
    # c4 as specified (the plain weights of c2) with the tower in int8 instead of e4m3
    "c4p": Config("c4p", 19, 20, 128, 0, 0, 3, 4096, (0, 80), (0, 80), 20260941, 9370002, weights_like="c2"),
    # c4 as specified (plain weights of c2, e4m3 weights and activations) with every operand carried as a pair of
    # e4m3 numbers, value and remainder (precision code 4), and with pairs for the activations only (code 5)
    "c4x": Config("c4x", 19, 20, 128, 0, 0, 4, 4096, (0, 80), (0, 80), 20260941, 9370002, weights_like="c2"),
    "c4a": Config("c4a", 19, 20, 128, 0, 0, 5, 4096, (0, 80), (0, 80), 20260941, 9370002, weights_like="c2"),
    "c5": Config("c5", 112, 40, 256, 1, 1, 1, 1024, (0, 80), (0, 80), 20260942, 9370005,
                 sweep=(16, 64, 256, 1024, 4096, 8192)),
}

# 512 positions, drawn with the config's own ply ranges, that fix the head scales (and, for the
# FP8 tower, the activation scales).  A separate seed keeps them disjoint from the test batches.
CALIBRATION_SEED_OFFSET = 777_000_000
CALIBRATION_COUNT = 512


def tiny_config(name="tiny", in_planes=19, blocks=2, channels=16, policy_head=0, value_head=0,
                precision=0, batch=8, weight_seed=4242) -> Config:
    """A small net for tests that need the oracle to finish at once."""
    return Config(name, in_planes, blocks, channels, policy_head, value_head, precision, batch,
                  (0, 80), (0, 80), 20260900, weight_seed)
