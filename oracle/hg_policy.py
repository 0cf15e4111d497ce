"""Plain-Python statements of the paper's host-side policy pieces.  TEST INFRASTRUCTURE ONLY (see
``hg_oracle.py``): the product's C++ versions are checked against these.

* feedback_scheduler_step: Algorithm 1, one evaluation of its if/else on carried (K, strategy), branch for
  branch as the listing has them.  Readings where the listing is silent: "increase"/"decrease" move K by a
  fixed step within [K_min, K_max].  The listing's first branch raises K whatever the strategy is and no
  branch ever sets the strategy back, so the switch to Pre-QK^T is one-way within a run (the offloaded
  context only grows, and with it the cost of Post-QK^T): in Pre-QK^T mode K keeps tracking the balance
  point T_cpu + T_tx = T_gpu.
* topk: Post-QK^T selection (Section 4.3): the K largest scores; ties to the lower index.
* positions: a position-based Pre-QK^T selection (Section 4.5): first `sinks` and last `window` tokens.
* ranked: Pre-QK^T selection from ranked candidate lists (Section 4.5), one list per KV head of a sequence:
  every head takes the same number of leading entries, as many as K, the host token count and the shortest
  list allow.
"""
POST_QK, PRE_QK = 0, 1


def feedback_scheduler_init(k_min):
    return k_min, POST_QK                                   # Initialize K <- K_min, strategy <- Post-QK^T


def feedback_scheduler_step(k, strategy, t_gpu, t_cpu, t_tx, k_min, k_max, step):
    if t_cpu + t_tx <= t_gpu:                               # CPU stage hidden behind the GPU stage
        k = min(k_max, k + step)                            # increase K to improve accuracy
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


def ranked(lists, k, n_host):
    """lists: one ranked list of host token indices per KV head of a sequence (-1 padded).  Returns the entries
    each head takes."""
    def valid_prefix(lst):
        n = 0
        for t in lst:
            if t < 0 or t >= n_host:
                break
            n += 1
        return n
    n = min([k, n_host] + [valid_prefix(l) for l in lists])
    return [list(l[:n]) for l in lists]
