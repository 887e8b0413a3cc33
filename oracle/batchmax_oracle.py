"""Plain fp64 CPU oracle for attention with KV-cache eviction during prefilling
and decoding (Batch-Max, Sec. 3: Algorithm 1 + the average-attention rule).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the
benchmark's CPU-baseline leg.  It is slow on purpose, takes the algorithm's
steps in the paper's order, and shares nothing with the CUDA path.

The method is a heuristic whose result depends on the whole history of
evictions, so the oracle *is* the algorithm, one step after the other, for one
independent (layer, sample, kv-head) cache ("for each attention head and
sample", Sec. 3.2).  All arithmetic is float64.

Readings of points the paper leaves open (each is a convention of this build):
  * "attention weights" are the post-softmax probabilities of causal scaled
    dot-product attention with scale 1/sqrt(d) (Sec. 3.2 uses weights/scores
    interchangeably).
  * grouped-query attention (not mentioned in the paper): one cache and one
    sum_weights vector per KV head; the weights of the g query heads of the
    group are added, and ave_weights is divided by g so it stays in [0, 1].
  * the denominator of ave_weights is the exact number of attention rows that
    were accumulated for the pair, curr_id + 1 - kv_ids with curr_id the last
    position processed (the justification given in Sec. 3.2, second paragraph).
    Algorithm 1's literal decode-time curr_id (one larger) is available through
    the ``curr_id`` argument of :meth:`UnitCache.evict`.
  * ties in ave_weights: the pair with the lower position id is kept.
  * left padding (Sec. 3: shorter prompts are padded on the left): a padding
    position produces no attention row (its output is zero and it adds nothing
    to sum_weights) and its pair is masked for every query, so its sum_weights
    stays 0; padding pairs rank below every real pair at an eviction (the paper
    does not say how padding meets eviction).
  * survivors keep their sum_weights (the vector is "variable-sized": entries
    leave with their pairs and nothing is reset).

The extreme decoding-only comparison of Algorithm 3 (keep only the most recent
pair) is here as well, :meth:`UnitCache.keep_most_recent` and
:func:`run_extreme_decoding`, because the library's timed comparison arm is
checked against it.

Four rules of other methods, as far as Sec. 2 describes them, can replace the
average (``rule=`` of :class:`UnitCache`): "sum_recent" (H2O), "current_query"
(TOVA), "window_pooled" (SnapKV) and "average_std" (RoCo); their parameters the
paper does not give are arguments here (see :meth:`UnitCache.ranking_scores`).

Parity unpinned (conventions, not derivable from the paper): the GQA sum, the
tie direction and the denominator reading above.  Everything else is pinned by
tests/test_oracle_pins.py.
"""
from __future__ import annotations

import math

import numpy as np


class UnitCache:
    """KV cache of one (layer, sample, kv-head) with the eviction state of
    Sec. 3.2: ``kv_ids`` (position ids, ascending), ``sum_weights`` and the
    key/value rows themselves."""

    RULES = ("average", "sum_recent", "current_query", "window_pooled", "average_std")

    def __init__(self, d: int, g: int = 1, scale: float | None = None, left_pad: int = 0,
                 rule: str = "average", window: int = 32, pool: int = 7, std_share: float = 0.5):
        assert rule in self.RULES
        self.rule = rule
        self.window = int(window)        # window_pooled: queries observed / recent pairs kept (Sec. 2, SnapKV's w)
        self.pool = int(pool)            # window_pooled: width of the max-pooling over neighbouring positions (odd)
        self.std_share = float(std_share)  # average_std: share of the kept pairs chosen by standard deviation
        assert self.window >= 1 and self.pool >= 1 and self.pool % 2 == 1 and 0.0 <= self.std_share <= 1.0
        assert not (rule == "average_std" and left_pad > 0), "average_std is defined without left padding here"
        self.d = int(d)
        self.g = int(g)
        self.left_pad = int(left_pad)  # positions 0 .. left_pad-1 of this sample are padding (Sec. 3)
        self.scale = (1.0 / math.sqrt(d)) if scale is None else float(scale)
        self.kv_ids = np.zeros(0, dtype=np.int64)
        self.k = np.zeros((0, d), dtype=np.float64)
        self.v = np.zeros((0, d), dtype=np.float64)
        self.sum_weights = np.zeros(0, dtype=np.float64)
        self.sum_sq = np.zeros(0, dtype=np.float64)   # sum of squared attention weights (average_std only)
        self.last_pos = -1            # curr_id: last position id processed
        self.evicted_mass = 0.0       # sum_weights that left with evicted pairs
        self.rows_processed = 0       # number of attention rows accumulated (queries x g)
        self.last_eviction = None     # snapshot of the most recent eviction

    def __len__(self) -> int:
        return int(self.kv_ids.shape[0])

    # ------------------------------------------------------------------ Sec. 3.2, update equation
    def process_block(self, q, k, v, pos0: int, evict_to: int = -1, return_weights: bool = False):
        """Forward pass with a block of ``I`` inputs at positions pos0..pos0+I-1.

        q: (I, g, d)   k, v: (I, d).  Returns the attention output (I, g, d).
        Every query attends to all cached pairs and to the block's pairs at
        positions <= its own; sum_weights += sum_i attn_weights[i] (Sec. 3.2);
        new pairs start from a zero sum_weights entry.  If ``evict_to >= 0``
        and the cache is larger afterwards, it is cut back to ``evict_to``.
        """
        q = np.asarray(q, dtype=np.float64)
        k = np.asarray(k, dtype=np.float64)
        v = np.asarray(v, dtype=np.float64)
        I = q.shape[0]
        assert q.shape == (I, self.g, self.d) and k.shape == (I, self.d) and v.shape == (I, self.d)
        if pos0 != self.last_pos + 1:
            raise ValueError(f"pos0={pos0} does not follow last position {self.last_pos}")
        n_old = len(self)
        self.kv_ids = np.concatenate([self.kv_ids, pos0 + np.arange(I, dtype=np.int64)])
        self.k = np.concatenate([self.k, k], axis=0)
        self.v = np.concatenate([self.v, v], axis=0)
        self.sum_weights = np.concatenate([self.sum_weights, np.zeros(I)])
        self.sum_sq = np.concatenate([self.sum_sq, np.zeros(I)])

        out = np.zeros((I, self.g, self.d))
        weights = np.zeros((I, self.g, n_old + I)) if return_weights else None
        real = self.kv_ids >= self.left_pad          # padding pairs are masked for every query
        n_real_queries = 0
        # rules that look at recent queries only: the weights of the block's last query (current_query) or of its
        # last `window` inputs (window_pooled) count, and nothing is carried over from earlier passes (Sec. 2)
        first_counted = {"current_query": I - 1, "window_pooled": I - min(self.window, I)}.get(self.rule, 0)
        if self.rule in ("current_query", "window_pooled"):
            self.sum_weights[:] = 0.0
        for i in range(I):
            if pos0 + i < self.left_pad:
                continue                             # a padding position: no output, no attention row
            n_real_queries += 1
            # visible pairs: every cached one, and the block's own up to position pos0 + i
            # (kv_ids is ascending, so these are the first m entries), minus the padding pairs.
            m = n_old + i + 1
            assert self.kv_ids[m - 1] == pos0 + i
            vis = slice(0, m) if self.left_pad == 0 else np.nonzero(real[:m])[0]
            for h in range(self.g):
                logits = self.scale * (self.k[vis] @ q[i, h])
                w = np.exp(logits - logits.max())
                w = w / w.sum()                      # attn_weights[i] for this head
                out[i, h] = w @ self.v[vis]
                if i >= first_counted:
                    self.sum_weights[vis] += w       # sum_weights += attn_weights[i]
                    if self.rule == "average_std":
                        self.sum_sq[vis] += w * w
                if return_weights:
                    weights[i, h, vis] = w
        self.last_pos = pos0 + I - 1
        self.rows_processed += n_real_queries * self.g
        if evict_to >= 0 and len(self) > evict_to:
            self.evict(evict_to)
        return (out, weights) if return_weights else out

    def decode_step(self, q, k, v, evict_to: int = -1):
        """One generated token: a block with I = 1 (Sec. 3.2: "during decoding I = 1").
        q: (g, d), k, v: (d,).  Returns (g, d)."""
        q = np.asarray(q, dtype=np.float64)[None]
        k = np.asarray(k, dtype=np.float64)[None]
        v = np.asarray(v, dtype=np.float64)[None]
        return self.process_block(q, k, v, self.last_pos + 1, evict_to)[0]

    # ------------------------------------------------------------------ Sec. 3.2, eviction rule
    def ave_weights(self, curr_id: int | None = None):
        """ave_weights = sum_weights / (curr_id + 1 - kv_ids), element-wise; divided by the
        group size so a GQA group's summed weights stay in [0, 1]."""
        curr_id = self.last_pos if curr_id is None else curr_id
        count = curr_id + 1 - self.kv_ids
        return self.sum_weights / (self.g * count)

    def ranking_scores(self, target: int, curr_id: int | None = None):
        """The value pairs are ranked by at an eviction down to ``target``.
        average: ave_weights (Sec. 3.2, the method's rule).
        sum_recent: the rule Sec. 2 ascribes to H2O -- the cache is split evenly between a window of the most
          recent pairs and the pairs with the largest sum of past attention weights: the floor(target / 2) most
          recent pairs rank first (+inf), the others by their raw sum_weights.
        current_query: the rule Sec. 2 ascribes to TOVA -- the weights of the current query alone (sum_weights
          holds nothing else under this rule, see process_block).
        window_pooled: the rule Sec. 2 ascribes to SnapKV -- a window of recent pairs stays (the min(window, target)
          most recent candidates, +inf); the others are ranked by the attention weights summed over the last
          `window` queries (what sum_weights holds under this rule), each replaced by the maximum over the `pool`
          neighbouring candidates centred on it (neighbours in cache order, the window excluded), so that kept
          positions come in runs rather than isolated.  Pooling by maximum and the two widths are this build's
          parameters: the paper names the pooling layer without describing it.
        average_std: the rule Sec. 2 / Sec. 3.2 ascribe to RoCo -- the kept pairs are split between the pairs whose
          attention weights have the largest standard deviation, floor(std_share * target) of them (+inf; ties to
          the lower position), and the largest average weights among the rest.  The standard deviation is over the
          g * (curr_id + 1 - kv_ids) weights the pair has received: sqrt(E[w^2] - E[w]^2).  The share is this
          build's parameter."""
        if self.rule == "average":
            return self.ave_weights(curr_id)
        if self.rule == "average_std":
            ave = self.ave_weights(curr_id)
            curr = self.last_pos if curr_id is None else curr_id
            cnt = self.g * (curr + 1 - self.kv_ids)
            std = np.sqrt(np.maximum(self.sum_sq / cnt - ave * ave, 0.0))
            n_std = int(math.floor(self.std_share * int(target) + 1e-9))
            protected = np.lexsort((self.kv_ids, -std))[:n_std]
            score = ave.copy()
            score[protected] = np.inf
            return score
        score = self.sum_weights.copy()
        if self.rule == "window_pooled":
            n = len(self)
            keep_recent = min(self.window, int(target))
            body = n - keep_recent                     # candidates outside the window of recent pairs
            half = self.pool // 2
            pooled = np.array([score[max(0, j - half):min(body, j + half + 1)].max() for j in range(body)])
            score[:body] = pooled
            score[body:] = np.inf
            score[self.kv_ids < self.left_pad] = 0.0
            return score
        if self.rule == "sum_recent":
            window = int(target) // 2
            if window > 0:
                score[len(self) - window:] = np.inf
            score[self.kv_ids < self.left_pad] = 0.0   # padding is never "recent": it ranks last whatever its position
        return score

    def evict(self, target: int, curr_id: int | None = None, kept_ids=None):
        """Remove the pairs with the smallest ave_weights until ``target`` remain.

        Ranking: ave_weights descending, ties -> lower position id first (padding pairs of a
        left-padded sample rank after every real pair); the first ``target``
        survive and stay in ascending position order (stable compaction).  ``kept_ids`` overrides
        the selection (used by lock-step parity to follow a choice made inside the tolerance
        band); the snapshot in ``last_eviction`` always holds the oracle's own choice.
        """
        n = len(self)
        target = int(target)
        if target >= n:
            return None
        ave = self.ranking_scores(target, curr_id)
        # primary: real pairs before padding pairs (padding always leaves first), then -score, then id
        order = np.lexsort((self.kv_ids, -ave, self.kv_ids < self.left_pad))
        own_keep = np.sort(order[:target])
        cut = float(ave[order[target - 1]]) if target > 0 else math.inf
        snap = {
            "cand_ids": self.kv_ids.copy(),
            "cand_ave": ave.copy(),
            "cand_sum_weights": self.sum_weights.copy(),
            "kept_ids": self.kv_ids[own_keep].copy(),
            "cut": cut,
            "target": target,
        }
        if kept_ids is None:
            keep = own_keep
        else:
            kept_ids = np.asarray(kept_ids, dtype=np.int64)
            assert kept_ids.shape[0] == target and np.all(np.diff(kept_ids) > 0)
            keep = np.searchsorted(self.kv_ids, kept_ids)
            assert np.array_equal(self.kv_ids[keep], kept_ids), "kept ids must be candidates"
        gone = np.ones(n, dtype=bool)
        gone[keep] = False
        self.evicted_mass += float(self.sum_weights[gone].sum())
        self.kv_ids = self.kv_ids[keep]
        self.k = self.k[keep]
        self.v = self.v[keep]
        self.sum_weights = self.sum_weights[keep]
        self.sum_sq = self.sum_sq[keep]
        self.last_eviction = snap
        return snap


    # ------------------------------------------------------------------ Algorithm 3's rule
    def keep_most_recent(self, keep: int = 1):
        """Remove all but the ``keep`` most recent pairs (the rule of the extreme decoding-only
        comparison, Algorithm 3, where keep = 1).  Survivors keep their sum_weights."""
        n = len(self)
        keep = int(keep)
        if keep >= n:
            return
        first = n - keep
        self.evicted_mass += float(self.sum_weights[:first].sum())
        self.kv_ids = self.kv_ids[first:]
        self.k = self.k[first:]
        self.v = self.v[first:]
        self.sum_weights = self.sum_weights[first:]
        self.sum_sq = self.sum_sq[first:]


# ---------------------------------------------------------------------- plain definition
def dense_causal_attention(q, k, v, scale: float | None = None):
    """Full-KV-cache attention (the no-eviction limit, "FKV" in Sec. 4), written out from the
    definition: out[i, h] = softmax_j<=i(scale * <q[i, h], k[j]>) . v.   q: (s, g, d), k, v: (s, d)."""
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    s, g, d = q.shape
    scale = 1.0 / math.sqrt(d) if scale is None else scale
    out = np.zeros((s, g, d))
    for i in range(s):
        for h in range(g):
            logits = np.array([scale * float(np.dot(q[i, h], k[j])) for j in range(i + 1)])
            w = np.exp(logits - logits.max())
            w /= w.sum()
            for j in range(i + 1):
                out[i, h] += w[j] * v[j]
    return out


# ---------------------------------------------------------------------- schedules
def _trace_entry(unit: UnitCache):
    return unit.kv_ids.copy()


def run_north_star(q, k, v, s: int, block: int, kv_max: int, steps: int, p_dec: int = 1,
                   g: int | None = None, scale: float | None = None, left_pad: int = 0, rule: str = "average",
                   **rule_params):
    """Blocks of ``block`` prompt tokens (ragged tail allowed), the cache cut back to ``kv_max``
    after every block; then ``steps`` decode steps, cut back to ``kv_max`` whenever the cache
    has grown to ``kv_max + p_dec``.   q: (s+steps, g, d); k, v: (s+steps, d); the first
    ``left_pad`` positions are padding.
    Returns (outputs (s+steps, g, d), trace of kv_ids after every call, unit)."""
    q = np.asarray(q, dtype=np.float64)
    g = q.shape[1] if g is None else g
    unit = UnitCache(q.shape[2], g, scale, left_pad, rule, **rule_params)
    outs, trace = [], []
    pos = 0
    while pos < s:
        I = min(block, s - pos)
        outs.append(unit.process_block(q[pos:pos + I], k[pos:pos + I], v[pos:pos + I], pos, kv_max))
        trace.append(_trace_entry(unit))
        pos += I
    for t in range(steps):
        full = len(unit) + 1 >= kv_max + p_dec
        outs.append(unit.decode_step(q[s + t], k[s + t], v[s + t], kv_max if full else -1)[None])
        trace.append(_trace_entry(unit))
    return np.concatenate(outs, axis=0), trace, unit


def cadence_algorithm1(prompt: int, limit: int, p: int, generated: int):
    """Algorithm 1 as a table of calls (op, first position, inputs, argument): the cache may reach ``limit`` pairs;
    whenever it would grow past it, ``p`` pairs leave first.  The prompt's first min(prompt, limit) tokens go in
    one block, the rest in blocks of at most ``p``; ``generated`` tokens mean ``generated - 1`` decode passes
    (prefilling emits the first new token), each at position prompt + pass index.  Ops: "block" (argument unused),
    "cut" (argument = pairs to keep; flagged when it happens inside the decode phase)."""
    calls, n = [], 0
    first = min(prompt, limit)
    calls.append(("block", 0, first, None))
    n, done = first, first
    while done < prompt:
        calls.append(("cut", 0, 0, (n - p, False)))
        n -= p
        take = min(p, prompt - done)
        calls.append(("block", done, take, None))
        n, done = n + take, done + take
    for step in range(generated - 1):
        if n == limit:
            calls.append(("cut", 0, 0, (n - p, True)))
            n -= p
        calls.append(("block", prompt + step, 1, None))
        n += 1
    return calls


def cadence_extreme_decoding(prompt: int, limit: int, generated: int, block: int | None = None):
    """Algorithm 3 as a table of calls: the whole prompt with a full cache (in blocks of ``block`` positions when
    given), then only the newest pair survives; each of the ``generated - 1`` decode passes appends one pair, and a
    cache that has grown to ``limit`` pairs is cut back to its newest pair.  Ops: "block", "newest" (argument =
    pairs to keep)."""
    calls = []
    block = prompt if block is None else block
    for pos in range(0, prompt, block):
        calls.append(("block", pos, min(block, prompt - pos), None))
    calls.append(("newest", 0, 0, 1))
    n = 1
    for step in range(generated - 1):
        calls.append(("block", prompt + step, 1, None))
        n += 1
        if n == limit:
            calls.append(("newest", 0, 0, 1))
            n = 1
    return calls


def run_cadence(q, k, v, calls, scale: float | None = None, decode_denominator_plus_one: bool = False):
    """Feeds a table of calls to one cache.  Returns (outputs of every block in order, kv_ids after every block,
    the cache, cache sizes: after every "cut" and after every decode block that follows a "newest")."""
    q = np.asarray(q, dtype=np.float64)
    unit = UnitCache(q.shape[2], q.shape[1], scale)
    outs, trace, sizes = [], [], []
    seen_newest = False
    for op, pos0, I, arg in calls:
        if op == "block":
            outs.append(unit.process_block(q[pos0:pos0 + I], k[pos0:pos0 + I], v[pos0:pos0 + I], pos0))
            trace.append(_trace_entry(unit))
            if seen_newest:
                sizes.append(len(unit))
        elif op == "cut":
            keep, in_decode = arg
            # the position about to be processed, not yet attended: one more than the rows accumulated
            curr = unit.last_pos + 1 if (in_decode and decode_denominator_plus_one) else None
            unit.evict(keep, curr_id=curr)
            sizes.append(len(unit))
        elif op == "newest":
            unit.keep_most_recent(arg)
            seen_newest = True
        else:
            raise ValueError(op)
    return np.concatenate(outs, axis=0), trace, unit, sizes


def run_algorithm1(q, k, v, s: int, kv_bar: int, p: int, max_gen: int, scale: float | None = None,
                   literal_decode_curr_id: bool = False):
    """Algorithm 1 (see :func:`cadence_algorithm1`).  ``literal_decode_curr_id``: at a removal inside the decode
    loop use the printed decode-time curr_id (the position about to be generated, one more than the rows
    accumulated) in the rule's denominator instead of this build's reading.
    Returns (outputs, kv_ids after every block, cache, sizes after every removal)."""
    return run_cadence(q, k, v, cadence_algorithm1(s, kv_bar, p, max_gen), scale, literal_decode_curr_id)


def run_decode_only(q, k, v, s: int, block: int, kv_max: int, steps: int, p_dec: int = 1,
                    scale: float | None = None):
    """Decoding-only compression (Sec. 1): the whole prompt is cached during prefilling (processed
    here in blocks of ``block`` with no eviction), the cache is compressed to ``kv_max`` once after
    the prompt, then decoding proceeds as in :func:`run_north_star`."""
    q = np.asarray(q, dtype=np.float64)
    unit = UnitCache(q.shape[2], q.shape[1], scale)
    outs, trace = [], []
    pos = 0
    while pos < s:
        I = min(block, s - pos)
        outs.append(unit.process_block(q[pos:pos + I], k[pos:pos + I], v[pos:pos + I], pos))
        pos += I
    unit.evict(kv_max)
    trace.append(_trace_entry(unit))
    for t in range(steps):
        full = len(unit) + 1 >= kv_max + p_dec
        outs.append(unit.decode_step(q[s + t], k[s + t], v[s + t], kv_max if full else -1)[None])
        trace.append(_trace_entry(unit))
    return np.concatenate(outs, axis=0), trace, unit


def run_extreme_decoding(q, k, v, s: int, kv_bar: int, max_gen: int, block: int | None = None,
                         scale: float | None = None):
    """Algorithm 3, extreme decoding-only eviction (see :func:`cadence_extreme_decoding`).
    Returns (outputs, cache, cache size after every decode pass)."""
    out, _, unit, sizes = run_cadence(q, k, v, cadence_extreme_decoding(s, kv_bar, max_gen, block), scale)
    return out, unit, sizes
