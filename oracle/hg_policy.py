"""Plain-Python statements of the paper's host-side policy pieces.  TEST INFRASTRUCTURE ONLY (see
``hg_oracle.py``): the product's C++ versions are checked against these.

* feedback_scheduler_step: Algorithm 1, one evaluation of its if/else on carried (K, strategy).
  Readings where the listing is silent: "increase"/"decrease" move K by a fixed step within
  [K_min, K_max]; when the CPU stage is hidden again while in Pre-QK^T, the strategy first goes back to
  Post-QK^T (the listing's initial, accuracy-friendly mode) before K grows.
* topk: Post-QK^T selection (Section 4.3): the K largest scores; ties to the lower index.
* positions: a position-based Pre-QK^T selection (Section 4.5): first `sinks` and last `window` tokens.
"""
POST_QK, PRE_QK = 0, 1


def feedback_scheduler_init(k_min):
    return k_min, POST_QK                                   # Initialize K <- K_min, strategy <- Post-QK^T


def feedback_scheduler_step(k, strategy, t_gpu, t_cpu, t_tx, k_min, k_max, step):
    if t_cpu + t_tx <= t_gpu:                               # CPU stage hidden behind the GPU stage
        if strategy == PRE_QK:
            strategy = POST_QK
        else:
            k = min(k_max, k + step)                        # increase K to improve accuracy
    else:
        if k > k_min:
            k = max(k_min, k - step)                        # decrease K while ensuring K >= K_min
        else:
            strategy = PRE_QK
    return k, strategy


def topk(scores, k):
    order = sorted((i for i, s in enumerate(scores) if s == s), key=lambda i: (-scores[i], i))
    return sorted(order[:k])


def positions(n_tokens, sinks, window, k):
    sinks = max(0, min(sinks, n_tokens))
    window = max(0, min(window, n_tokens - sinks))
    ns = min(sinks, k)
    nw = min(window, k - ns)
    return list(range(ns)) + list(range(n_tokens - nw, n_tokens))
