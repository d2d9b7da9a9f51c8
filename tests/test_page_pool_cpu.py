"""The page pool's host-side decisions (no GPU): the library's bookkeeping against a model of
the sharing rules written here."""
import pytest

from paper_2505_13544_b200 import binding as M
from paper_2505_13544_b200 import synth

PAGE = 64


class ModelPool:
    """Reference model: a page is identified by its content history, so two sequences share a
    page exactly when the library is allowed to let them (same parent, page not written since).
    Sequences are lists of page objects; a page object is shared by reference."""

    def __init__(self):
        self.seqs = {}

    def prepare(self, seq, n_slots, write_slot):
        pages = self.seqs.setdefault(seq, [])
        copies = 0
        while len(pages) * PAGE < n_slots:
            pages.append(object())
        if write_slot >= 0:
            k = write_slot // PAGE
            shared = sum(1 for other in self.seqs.values() for pg in other if pg is pages[k]) > 1
            if shared:
                pages[k] = object()
                copies = 1 if write_slot % PAGE > 0 else 0
        return copies

    def reorder(self, parents):
        old = self.seqs
        self.seqs = {b: list(old.get(p, [])) for b, p in enumerate(parents)}

    def in_use(self):
        return len({id(pg) for pages in self.seqs.values() for pg in pages})

    def sharing(self):
        """Partition of (seq, index) entries by page identity."""
        groups = {}
        for b, pages in self.seqs.items():
            for k, pg in enumerate(pages):
                groups.setdefault(id(pg), []).append((b, k))
        return sorted(sorted(v) for v in groups.values())


def library_sharing(pool, n_seqs):
    groups = {}
    for b in range(n_seqs):
        for k, pg in enumerate(pool.row(b)):
            groups.setdefault(pg, []).append((b, k))
    return sorted(sorted(v) for v in groups.values())


@pytest.mark.parametrize("stride,beam,n_utt", [(2, 4, 3), (1, 3, 2), (3, 5, 1)])
def test_pool_follows_the_sharing_rules(stride, beam, n_utt):
    n_seq = beam * n_utt
    pool = M.PagePool(n_pages=4096, max_seqs=n_seq, max_pages_per_seq=16)
    model = ModelPool()
    lengths = synth.ragged_lengths(11, n_utt, 1, 5 * PAGE * stride // 2)
    tokens = []
    for u, t in enumerate(lengths):          # every hypothesis of an utterance starts from its prompt
        for k in range(beam):
            b = u * beam + k
            n_slots = -(-t // stride)
            assert pool.prepare(b, n_slots, -1) == []
            assert model.prepare(b, n_slots, -1) == 0
            tokens.append(t)
    try:
        for step in range(3 * PAGE):
            for b in range(n_seq):
                slot = tokens[b] // stride
                copies = pool.prepare(b, slot + 1, slot)
                want = model.prepare(b, slot + 1, slot)
                assert len(copies) == want
                for src, dst, rows in copies:
                    assert rows == slot % PAGE and src != dst
                    assert dst == pool.row(b)[slot // PAGE]
                tokens[b] += 1
            assert pool.in_use() == model.in_use()
            assert library_sharing(pool, n_seq) == model.sharing()
            parents = synth.beam_parents(5, step, n_utt, beam)
            pool.reorder(parents, n_seq)
            model.reorder(parents)
            tokens = [tokens[p] for p in parents]
            assert pool.in_use() == model.in_use()
            assert library_sharing(pool, n_seq) == model.sharing()
            for groups in model.sharing():
                page = pool.row(groups[0][0])[groups[0][1]]
                assert pool.ref(page) == len(groups)
    finally:
        pool.close()


def test_pool_exhaustion_leaves_the_state_unchanged():
    pool = M.PagePool(n_pages=3, max_seqs=2, max_pages_per_seq=4)
    try:
        assert pool.prepare(0, 2 * PAGE, -1) == []
        with pytest.raises(M.MTLAError) as err:
            pool.prepare(1, 2 * PAGE, -1)
        assert err.value.status == -4
        assert pool.in_use() == 2 and pool.row(1) == []
        assert pool.prepare(1, PAGE, -1) == []
        assert pool.in_use() == 3
        pool.reorder([1], 2)                   # sequence 0 is dropped: its pages come back
        assert pool.in_use() == 1
        assert pool.prepare(0, 2 * PAGE + 1, 2 * PAGE) == []   # the batch is one sequence now
        assert pool.in_use() == 3
    finally:
        pool.close()
