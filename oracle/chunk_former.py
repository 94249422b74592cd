"""TEST INFRASTRUCTURE — plain restatement of the token-wise chunk former (Section 3.1).

Only tests, the smoke check and the bench's cpu_baseline / reference arm may import this
module.  It shares no code with the C++ scheduler front and does not import it.

What Section 3.1 fixes: every step takes a fixed budget of tokens from the scheduling queues to
form one chunk that may mix prefill, decode and verify tokens; prefill is prioritised; a prompt
longer than the space left is split so the chunk stays within the budget; some slots are
reserved for decode and speculative tokens; a prefill-only chunk is formed only when no decode or
speculative tokens are waiting; under low load a chunk may be smaller than the budget.

What it leaves open, and the reading taken here (parity unpinned against the paper: it prints no
worked example of a chunk; pinned by invariants, brute force on small streams and a hand-worked
example of this reading):
  * queues: one FIFO of prefill requests (remaining prompt tokens after the prefix-cache match)
    and one FIFO shared by decode (1 token) and verify (a whole token tree) entries;
  * step 1: decode / verify entries are taken from the head of their FIFO while their tokens fit
    into the reserved slots R — except that the head entry is always taken when the reserved
    slots are still empty (a tree larger than R must not starve);
  * step 2: prefill requests are taken in order into the space left (budget minus step 1), the
    head request contributing min(remaining prompt, space) tokens; a request that is not
    finished stays at the head with its kvLen advanced by what was scheduled;
  * step 3: if space is still left (the prefill queue ran dry), further decode / verify entries
    are taken in order while they fit;
  * an entry is never split or reordered within its queue; a chunk holds at most `max_requests`
    entries; the chunk lists its prefill parts first, then the decode / verify entries.
"""
from __future__ import annotations

from collections import deque
from typing import List, Optional, Sequence, Tuple

KIND_PREFILL, KIND_DECODE, KIND_VERIFY = 0, 1, 2


class ChunkFormer:
    def __init__(self, budget: int, reserved_dv: int, max_requests: int):
        assert budget >= 1 and 0 <= reserved_dv <= budget and max_requests >= 1
        self.budget, self.reserved, self.max_requests = budget, reserved_dv, max_requests
        self.prefill = deque()  # [id, remaining, kv_len]
        self.dv = deque()       # (id, kind, kv_len, tokens, parents or None)

    def add_prefill(self, rid: int, prompt_tokens: int, cached_tokens: int) -> None:
        assert 0 <= cached_tokens < prompt_tokens
        self.prefill.append([rid, prompt_tokens - cached_tokens, cached_tokens])

    def add_decode(self, rid: int, kv_len: int) -> None:
        assert kv_len >= 0
        self.dv.append((rid, KIND_DECODE, kv_len, 1, None))

    def add_verify(self, rid: int, kv_len: int, parents: Sequence[int]) -> None:
        n = len(parents)
        assert 1 <= n <= self.budget and kv_len >= 0
        self.dv.append((rid, KIND_VERIFY, kv_len, n, list(parents)))

    def pending(self) -> Tuple[int, int]:
        return sum(p[1] for p in self.prefill), sum(e[3] for e in self.dv)

    def next_chunk(self) -> List[dict]:
        """Entries of the next chunk: dicts with id, kind, q_len, kv_len, last (prefill: the prompt
        is complete with this part), parents (verify).  Empty when nothing is queued."""
        taken_dv: List[tuple] = []
        used = 0
        # step 1: reserved slots
        while self.dv and len(taken_dv) < self.max_requests:
            tokens = self.dv[0][3]
            if used + tokens <= self.reserved or (used == 0 and tokens <= self.budget):
                taken_dv.append(self.dv.popleft())
                used += tokens
                if used >= self.reserved:
                    break
            else:
                break
        # step 2: prefill into the space left
        parts: List[dict] = []
        while self.prefill and used < self.budget and len(parts) + len(taken_dv) < self.max_requests:
            head = self.prefill[0]
            take = min(head[1], self.budget - used)
            parts.append(dict(id=head[0], kind=KIND_PREFILL, q_len=take, kv_len=head[2],
                              last=take == head[1], parents=None))
            head[1] -= take
            head[2] += take
            used += take
            if head[1] == 0:
                self.prefill.popleft()
        # step 3: leftover space goes to further decode / verify entries
        if not self.prefill:
            while self.dv and len(parts) + len(taken_dv) < self.max_requests:
                tokens = self.dv[0][3]
                if used + tokens > self.budget:
                    break
                taken_dv.append(self.dv.popleft())
                used += tokens
        out = parts
        for rid, kind, kv_len, tokens, parents in taken_dv:
            out.append(dict(id=rid, kind=kind, q_len=tokens, kv_len=kv_len, last=True, parents=parents))
        return out
