"""Memory accounting of App. A ("Calculation of memory saved from RAD") and Table 1.

TEST INFRASTRUCTURE ONLY.  The paper's rule, restated: the baseline keeps
every input of a linear or convolution layer at 32 bits per entry and the
softmax input; RAD keeps ceil(fraction * d) entries of each such input at 32
bits, the whole softmax input, and one bit per entry of every ReLU output;
average pooling and biases need nothing.  Table 1 is per-element bytes times
the minibatch size (150) plus the weights, in units of 10^6 bytes.
"""
import math

BATCH = 150

# (inputs of sampled layers, softmax input, ReLU-bit counts as the paper prints them, parameters)
PAPER_NETS = {
    # 784-300-300-300-10 MLP
    "mlp": dict(sampled=[784, 300, 300, 300], logits=10, relu_bits=[300, 300, 300],
                params=(784 * 300 + 300) + 2 * (300 * 300 + 300) + (300 * 10 + 10), extra=0),
    # 5x5 conv 16/32/32/32 with two 2x2 average pools, FC-10; the ReLU-bit
    # counts are the ones the paper prints (second and fourth are post-pool sizes)
    "cnn": dict(sampled=[3 * 32 * 32, 16 * 32 * 32, 32 * 16 * 16, 32 * 16 * 16, 32 * 8 * 8],
                logits=10, relu_bits=[16384, 8192, 8192, 2048],
                params=(75 * 16 + 16) + (400 * 32 + 32) + 2 * (800 * 32 + 32) + (2048 * 10 + 10),
                extra=0),
    # IRNN, 784 steps, hidden 100: per step the scalar input and the previous
    # hidden state, plus the last hidden state and the softmax input.  Table 1's
    # row is matched only with a constant 784*100*4 bytes on top of the
    # weights, whose origin the paper does not state.
    "rnn": dict(sampled=[1, 100] * 784 + [100], logits=10, relu_bits=[100] * 784,
                params=(100 + 100) + (100 * 100 + 100) + (100 * 10 + 10), extra=784 * 100 * 4),
}


def per_element_bytes(net: str, fraction: float) -> float:
    n = PAPER_NETS[net]
    if fraction >= 1.0:
        return (sum(n["sampled"]) + n["logits"]) * 4.0
    kept = sum(math.ceil(round(fraction * d, 9)) for d in n["sampled"])
    return (kept + n["logits"]) * 4.0 + sum(n["relu_bits"]) / 8.0


def table1_megabytes(net: str, fraction: float) -> float:
    n = PAPER_NETS[net]
    return (per_element_bytes(net, fraction) * BATCH + n["params"] * 4 + n["extra"]) / 1e6
