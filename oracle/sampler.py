"""fp64 CPU oracle for the sampling-stage truncation (Sec. 3.4, last paragraph;
Fig. "whole procedure of one inference step", caption).

TEST INFRASTRUCTURE ONLY: only the tests, the smoke check and the CPU-baseline
leg of the benchmark may import this module.  It shares no code with the CUDA
path and imports nothing from it.

The paper cuts the model's output to the tokens of the current generation block
before sampling, so that the float softmax runs over L_b rows per sequence
instead of N.  What a confidence-based sampler of a block-wise diffusion LLM
needs from that softmax is, per block row, the most probable token and its
probability (rows above a confidence threshold are decoded in this step); the
log normaliser is returned as well.

Readings where the paper is silent: the softmax is over the whole vocabulary, in
float; among tokens of exactly equal logit the lowest token id is the most
probable one.

Plain definition, numpy in double precision: p_v = exp(x_v) / sum_u exp(x_u).
"""
import numpy as np


def block_confidence(logits, rows):
    """logits [T, V] (any float dtype; values as the model stores them), rows [n]
    indices of the current block's tokens.  Returns (token [n] int64, conf [n],
    lse [n]): argmax_v p_v (lowest id among ties), max_v p_v, log sum_v exp(x_v),
    each over row rows[i] only -- no other row of `logits` is looked at."""
    rows = np.asarray(rows, dtype=np.int64)
    n = rows.shape[0]
    token = np.zeros(n, dtype=np.int64)
    conf = np.zeros(n, dtype=np.float64)
    lse = np.zeros(n, dtype=np.float64)
    for i, r in enumerate(rows):
        x = np.asarray(logits[r], dtype=np.float64)
        e = np.exp(x - x.max())          # the shift cancels in the ratio; it only avoids overflow
        p = e / e.sum()
        token[i] = int(np.argmax(x == x.max()))   # exp is monotonic: the first index that attains the largest logit
        conf[i] = p[token[i]]
        lse[i] = np.log(e.sum()) + x.max()
    return token, conf, lse
