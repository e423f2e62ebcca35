"""TEST INFRASTRUCTURE ONLY: the server's request queue and batch planner, written out with plain lists.

Section 3.4 of the paper: requests of many devices wait in a queue; a batch planner takes requests out of it
and forwards one batch to the target model.  The paper's scheme is static batching (wait for a fixed number of
requests); continuous batching takes whatever has arrived.  The paper pads a batch to a common length; the
verification step here is ragged, so a step's capacity is counted in tokens, sum (k_i + 1).

Rules (the same for both policies unless stated):
  * requests leave the queue in arrival order;
  * a context is verified at most once per step: a later request of a context that is already in the batch
    stays queued, in place;
  * a request that does not fit the tokens left in the step ends the batch (nothing overtakes it);
  * static: a batch has at most batch_size requests and is not formed while fewer are available, unless the
    caller flushes or the step's token capacity is what ended the scan;
  * continuous: a batch has at most max_batch requests and is formed whenever anything waits.
"""
from __future__ import annotations

STATIC, CONTINUOUS = 0, 1


class PlannerModel:
    def __init__(self, policy: int, batch_size: int, max_batch: int, max_step_tokens: int):
        self.policy, self.batch_size, self.max_batch, self.max_step_tokens = policy, batch_size, max_batch, max_step_tokens
        self.queue = []          # (ticket, ctx, k) in arrival order

    def push(self, ticket: int, ctx: int, k: int) -> bool:
        if k < 0 or k + 1 > self.max_step_tokens:
            return False
        self.queue.append((ticket, ctx, k))
        return True

    def next_batch(self, flush: bool = False):
        limit = self.batch_size if self.policy == STATIC else self.max_batch
        chosen, contexts, tokens, full = [], set(), 0, False
        for pos, (ticket, ctx, k) in enumerate(self.queue):
            if len(chosen) == limit:
                break
            if ctx in contexts:
                continue
            if tokens + k + 1 > self.max_step_tokens:
                full = True
                break
            contexts.add(ctx)
            tokens += k + 1
            chosen.append(pos)
        if not chosen:
            return []
        if self.policy == STATIC and not flush and not full and len(chosen) < self.batch_size:
            return []
        out = [self.queue[p][0] for p in chosen]
        self.queue = [r for p, r in enumerate(self.queue) if p not in set(chosen)]
        return out


def attention_plan_end_time(n_keys, q_tokens, chunk_keys, n_kv_heads: int, group: int, resident_blocks: int) -> float:
    """How long the attention items of a cut take by the planner's model, in key-tile times: a request of n keys and
    q tokens costs ceil(n / 64) tiles, weighted 1.15 with more than 16 query rows (q * group) and 1.93 with more than
    32, once per 64 query rows; an item carries its share of that plus 6 when its request is cut and 3 when it is
    not; the items of one part (one per KV head) start side by side, costly-row requests first, then longest first,
    each on the group of blocks that is free earliest."""
    items = []
    for n, q, c in zip(n_keys, q_tokens, chunk_keys):
        rows = q * group
        weight = 1.93 if rows > 32 else 1.15 if rows > 16 else 1.0
        cost = -(-n // 64) * ((rows + 63) // 64) * weight
        parts = -(-n // c)
        for j in range(parts):
            count = min(c, n - j * c)
            items.append((rows > 32, cost * count / n + (6.0 if parts > 1 else 3.0)))
    items.sort(key=lambda it: (not it[0], -it[1]))
    free_at = [0.0] * max(1, resident_blocks // n_kv_heads)
    for _, w in items:
        k = free_at.index(min(free_at))
        free_at[k] += w
    return max(free_at)
