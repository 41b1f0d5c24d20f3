"""The rank rule of the adaptive configuration, stated with the library sort (numpy lexsort): an
independent third statement beside the oracle's qsort and the CUDA kernel's counting, used by the
tests as a pin of the oracle and as the feeder of the adaptive workload's bit-widths."""
import numpy as np


def by_library_sort(scores, n_fp16, n_8bit, n_4bit):
    """Tokens ordered by score, highest first, equal scores by lower index first; the first n_fp16
    keep FP16, the next n_8bit get 8 bits, the next n_4bit get 4 bits, the rest 2 bits."""
    scores = np.asarray(scores)
    n = scores.size
    order = np.lexsort((np.arange(n), -scores.astype(np.float64)))
    bits = np.empty(n, dtype=np.uint8)
    a, b, c = n_fp16, n_fp16 + n_8bit, n_fp16 + n_8bit + n_4bit
    bits[order[:a]] = 16
    bits[order[a:b]] = 8
    bits[order[b:c]] = 4
    bits[order[c:]] = 2
    return bits
