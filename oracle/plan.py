"""Index construction for a compaction event, restated in plain Python.

TEST INFRASTRUCTURE ONLY.  Follows the paper's Section 4 ("Snapshot &
partition": a history of |X| tokens becomes N = ceil(|X| / B) contiguous blocks,
the last one possibly short; "Dispatch": one sequence per block) and the paged
KV bookkeeping a serving engine keeps underneath (Section 4.2 names the engine;
the paper gives no detail, so the rules below are this library's own and are
stated in full):

* cu_seqlens      prefix sums of the block lengths
* pages           block b owns ceil((L_b + T) / P) pages, T = reserved summary
                  tokens; pages are dealt block by block, in order, from the
                  caller's free list
* slot of token p of block b:  page_indices[page_indptr[b] + p // P] * P + p % P
* prefill items   (block, q_tile) for q_tile < ceil(L_b / q_tile_rows); cost is
                  the number of keys its last row sees; order: descending cost,
                  ties by ascending block, then tile
* decode items    (block, kv_head, split): split s of block b covers pages
                  [s*C_b, min((s+1)*C_b, pages_b)); order: descending page count,
                  ties by ascending block, kv head, split.  C_b (pages per split)
                  is an input: one number for all blocks or one per block
* split_indptr    prefix sums of ceil(pages_b / C_b)
* chunked prefill (Section 4.2: the serving engine runs with chunked prefill enabled; the
                  paper gives no rule, this one is the library's reading) a block of L_b
                  tokens is prefilled in ceil(L_b / C) chunks of C tokens (the last one
                  short), a chunk every r steps, and decodes its T summary tokens in the T
                  steps after its last chunk's r steps; see mixed_schedule
* pages on demand (Section 8, "Dynamic block size and prompt selection": summaries of unknown
                  length) instead of reserving pages for T tokens per block, a block holds
                  pages for the tokens it has plus the next one; the rest of the free list is
                  a common reserve that any block draws from when it fills a page, and that a
                  finished block's pages go back to; see DynamicPages
* prefix-aware    (Section 4, "Prefix-aware target-at-end layout") each sequence
                  additionally starts with prefix_lens[b] cached history tokens in
                  shared pages: they come first in its page list, count in seq_lens,
                  in the cost of its prefill items and in its decode splits
"""
from __future__ import annotations

from typing import Dict, Sequence


def partition(history_len: int, block_size: int):
    """Section 4, step 1: N = ceil(|X| / B) contiguous blocks of B tokens."""
    if history_len < 1 or block_size < 1:
        raise ValueError("lengths must be positive")
    n = -(-history_len // block_size)
    lens = [block_size] * (n - 1)
    lens.append(history_len - block_size * (n - 1))
    return lens


def build_plan(block_lens: Sequence[int], max_new_tokens: int, page_size: int,
               free_pages: Sequence[int], num_kv_heads: int,
               q_tile_rows: int, pages_per_split, prefix_lens: Sequence[int] = (),
               shared_pages: Sequence[int] = (), shared_chunk_pages: int = 0) -> Dict[str, list]:
    """Independent chunks (no prefix_lens), or the prefix-aware layout of Section 4: sequence b
    (worker b) already has the first prefix_lens[b] tokens of the shared history cached in the first
    prefix_lens[b] / P entries of `shared_pages` (same pages for every worker: the prefix cache), and
    block_lens[b] are its own tokens (target block plus markers), stored after the prefix in pages of
    its own taken from the free list.  With shared_chunk_pages > 0 the decode of the shared pages is a
    scan of its own in chunks of that many pages: sequence b gets ceil(prefix pages / chunk) partial
    slots for it in front of the slots of its splits, and its splits cover its own pages only."""
    B = len(block_lens)
    prefix_lens = [int(x) for x in prefix_lens] if len(prefix_lens) else [0] * B
    if len(prefix_lens) != B or any(x < 0 or x % page_size for x in prefix_lens):
        raise ValueError("one page-aligned prefix length per block")
    if max(prefix_lens) > len(shared_pages) * page_size:
        raise ValueError("prefix longer than the shared pages")
    if B < 1:
        raise ValueError("need at least one block")
    if any(int(L) < 1 for L in block_lens):
        raise ValueError("block lengths must be >= 1")
    if isinstance(pages_per_split, int):
        pages_per_split = [pages_per_split] * B
    if len(pages_per_split) != B:
        raise ValueError("one split size per block")
    if max_new_tokens < 0 or page_size < 1 or q_tile_rows < 1 or min(pages_per_split) < 1:
        raise ValueError("bad parameter")

    cu = [0]
    for L in block_lens:
        cu.append(cu[-1] + int(L))

    pages_per_block, own_pages = [], []
    for b, L in enumerate(block_lens):
        tokens = int(L) + max_new_tokens
        own_pages.append((tokens + page_size - 1) // page_size)
        pages_per_block.append(prefix_lens[b] // page_size + own_pages[b])
    indptr = [0]
    for n in pages_per_block:
        indptr.append(indptr[-1] + n)
    if sum(own_pages) > len(free_pages):
        raise MemoryError("not enough free pages")
    page_indices, taken = [], 0
    for b in range(B):
        page_indices += [int(x) for x in shared_pages[: prefix_lens[b] // page_size]]
        page_indices += [int(free_pages[taken + i]) for i in range(own_pages[b])]
        taken += own_pages[b]

    slot_mapping = []
    for b, L in enumerate(block_lens):
        for p in range(prefix_lens[b], prefix_lens[b] + int(L)):
            page = page_indices[indptr[b] + p // page_size]
            slot_mapping.append(page * page_size + p % page_size)

    prefill = []
    for b, L in enumerate(block_lens):
        n_tiles = (int(L) + q_tile_rows - 1) // q_tile_rows
        for t in range(n_tiles):
            cost = prefix_lens[b] + min((t + 1) * q_tile_rows, int(L))
            prefill.append((-cost, b, t))
    prefill.sort()
    prefill_items = [[b, t] for (_, b, t) in prefill]

    split_indptr = [0]
    decode = []
    for b, n in enumerate(pages_per_block):
        c_b = int(pages_per_split[b])
        prefix_pages = prefix_lens[b] // page_size
        fixed = -(-prefix_pages // shared_chunk_pages) if shared_chunk_pages else 0
        if shared_chunk_pages:
            n -= prefix_pages                     # the splits cover the own pages only
        n_splits = (n + c_b - 1) // c_b
        split_indptr.append(split_indptr[-1] + fixed + n_splits)
        for g in range(num_kv_heads):
            for s in range(n_splits):
                size = min(c_b, n - s * c_b)
                decode.append((-size, b, g, s))
    decode.sort()
    decode_items = [[b, g, s] for (_, b, g, s) in decode]

    return {
        "cu_seqlens": cu,
        "page_indptr": indptr,
        "page_indices": page_indices,
        "seq_lens": list(prefix_lens),
        "slot_mapping": slot_mapping,
        "prefill_items": prefill_items,
        "decode_items": decode_items,
        "split_indptr": split_indptr,
    }


def mixed_schedule(block_lens: Sequence[int], chunk_tokens: int, max_new_tokens: int, decode_steps_per_chunk: int = 1):
    """Steps of one event with chunked prefill (Section 4.2: chunked prefill is enabled in the paper's
    serving engine, so a long block's prefill is cut into chunks that share steps with the decode of
    blocks that are already past their prefill; Section 6 is why it matters: 16k blocks are
    prefill-bound).  Rule, stated in full because the paper gives none (C = chunk_tokens,
    r = decode_steps_per_chunk: a chunk costs about as much as r decode steps, so the blocks that
    decode take r tokens while a chunk is prefilled beside them):

      chunk c of block b, rows [c*C, min((c+1)*C, L_b)), starts at step c*r, for c < n_b = ceil(L_b / C);
      block b decodes summary token t at step n_b*r + t, t = 0 .. T-1;
      the event has max_b(n_b)*r + T steps.

    Returns a list with one entry per step: {"prefill": [(block, first_row, rows)], "decode": [blocks]},
    both in ascending block order ("prefill" is empty in steps that start no chunk).
    """
    r = decode_steps_per_chunk
    if chunk_tokens < 1 or max_new_tokens < 0 or r < 1 or not len(block_lens) or any(int(L) < 1 for L in block_lens):
        raise ValueError("bad parameter")
    n_chunks = [-(-int(L) // chunk_tokens) for L in block_lens]
    steps = []
    for s in range(max(n_chunks) * r + max_new_tokens):
        pre = []
        if s % r == 0:
            c = s // r
            pre = [(b, c * chunk_tokens, min(chunk_tokens, int(L) - c * chunk_tokens))
                   for b, L in enumerate(block_lens) if c < n_chunks[b]]
        dec = [b for b in range(len(block_lens)) if n_chunks[b] * r <= s < n_chunks[b] * r + max_new_tokens]
        steps.append({"prefill": pre, "decode": dec})
    return steps


class DynamicPages:
    """Page bookkeeping when nothing is reserved for the summaries (the paper's Section 8 asks for
    per-block sizes that are not known in advance; the rule is this library's).

    A live block always holds exactly the pages for its cached tokens plus the next token:
    len // P + 1 pages (never more than its table holds, ceil((L + T) / P)).  It starts with that many
    from the front of the free list, block by block; the rest of the free list is the common reserve.
    A block that fills a page takes one page from the reserve; a finished block gives all its pages
    back.  WHICH page a block gets is free (concurrent blocks may draw in any order), so this class
    tracks counts, and `check` states what any valid outcome satisfies.
    """

    def __init__(self, block_lens: Sequence[int], max_new_tokens: int, page_size: int, free_pages: Sequence[int]):
        self.P = page_size
        self.len = [int(L) for L in block_lens]
        self.cap = [-(-(int(L) + max_new_tokens) // page_size) for L in block_lens]
        self.pages = [min(L // page_size + 1, c) for L, c in zip(self.len, self.cap)]
        if sum(self.pages) > len(free_pages):
            raise MemoryError("not enough free pages")
        self.all_pages = sorted(int(x) for x in free_pages)
        self.initial, taken = [], 0
        for n in self.pages:
            self.initial.append([int(x) for x in free_pages[taken:taken + n]])
            taken += n
        self.reserve = len(free_pages) - taken
        self.live = [True] * len(self.len)

    def step(self, active: Sequence[bool]) -> None:
        """One decode step: every active live block caches one token."""
        for b, a in enumerate(active):
            if not (a and self.live[b]):
                continue
            if self.len[b] // self.P >= self.pages[b]:
                raise MemoryError(f"block {b} has no page for its next token")
            self.len[b] += 1
            want = min(self.len[b] // self.P + 1, self.cap[b])
            if want > self.pages[b]:
                if self.reserve == 0:
                    continue            # stays short of a page; its next step fails
                self.reserve -= 1
                self.pages[b] += 1

    def release(self, blocks: Sequence[int]) -> None:
        for b in blocks:
            if self.live[b]:
                self.reserve += self.pages[b]
                self.pages[b] = 0
                self.live[b] = False

    def check(self, table_rows: Sequence[Sequence[int]], assigned: Sequence[int], lens: Sequence[int],
              ring: Sequence[int]) -> None:
        """table_rows[b][:assigned[b]] are block b's pages, `ring` the reserve's pages.  Raises
        AssertionError unless: counts and lengths are the model's; every page of the original free
        list is in exactly one place; a block's first pages are still the ones it started with."""
        assert list(lens) == self.len, ("lengths", list(lens), self.len)
        assert list(assigned) == self.pages, ("pages per block", list(assigned), self.pages)
        assert len(ring) == self.reserve, ("reserve", len(ring), self.reserve)
        held = [int(x) for b, row in enumerate(table_rows) for x in row[:assigned[b]]] + [int(x) for x in ring]
        assert sorted(held) == self.all_pages, "a page is lost, duplicated or foreign"
        for b, row in enumerate(table_rows):
            if self.live[b]:
                n = len(self.initial[b])
                assert [int(x) for x in row[:n]] == self.initial[b], f"block {b} lost its first pages"


def slot_of(plan: Dict[str, list], page_size: int, block: int, pos: int) -> int:
    """Pool slot (page * P + offset) of position `pos` of `block`."""
    page = plan["page_indices"][plan["page_indptr"][block] + pos // page_size]
    return page * page_size + pos % page_size
