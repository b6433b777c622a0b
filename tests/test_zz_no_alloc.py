"""vvs_decide_noalloc, the entry point for callers that are not allowed to allocate device memory
(their process handed the whole GPU to another allocator, or they sit in a loop that cannot
tolerate the synchronisation a cudaMalloc brings): its scratch is a fixed device array inside
the library instead of a context's arena.  It must give exactly what vvs_decide gives, also on a
second call that finds the first call's leftovers in the shared array, and it must refuse sizes
beyond the array's stated capacity.  Both entry points are also compared with the CPU oracle's
decision stage on the same probabilities.  Collected last on purpose (file name)."""
import numpy as np
import pytest

from test_gpu_decide import compare_exact, decide_case, gpu_decide, oracle_decide
from vvs_synth.configs import MODE_RELAXED, MODE_STRICT

pytestmark = pytest.mark.gpu


def _both(c, vb):
    rows, first_row, k, b = c["rows"], c["first_row"], c["n_draft_max"], c["n_images"]
    ctx = vb.vvs_create(vb.make_desc(c["ms"], b, rows, max(1, c["nbr_k"])))

    def with_ctx(d, o):
        if "row_ptr" in d:
            vb.vvs_bind_neighbors(ctx, d["row_ptr"], d["col"])
        vb.vvs_decide(ctx, target_probs=d["target_probs"], n_rows_per_seq=rows, first_row=first_row,
                      drafts=d["drafts"], n_images=b, n_draft_max=k, n_draft=d["n_draft"],
                      draft_probs=d["draft_probs"], uniforms=d["uniforms"], mode=c["mode"],
                      nbr_k=c["nbr_k"], delta=c["delta"], **o)

    import torch
    status = torch.zeros(1, dtype=torch.int32, device="cuda")

    def no_alloc(d, o):
        vb.vvs_decide_noalloc(status_bits=status, target_probs=d["target_probs"], vocab=c["ms"].vocab,
                              vocab_offset=c["ms"].vocab_offset, n_rows_per_seq=rows,
                              first_row=first_row, drafts=d["drafts"], n_images=b, n_draft_max=k,
                              n_draft=d["n_draft"], draft_probs=d["draft_probs"],
                              uniforms=d["uniforms"], nbr_row_ptr=d.get("row_ptr"),
                              nbr_col=d.get("col"), mode=c["mode"], nbr_k=c["nbr_k"],
                              delta=c["delta"], **o)
    want = gpu_decide(c, with_ctx)
    got = gpu_decide(c, no_alloc)
    assert int(status.item()) == 0          # the caller-owned status word: no device-side complaint
    vb.vvs_destroy(ctx)
    compare_exact(c, got, oracle_decide(c))  # the allocation-free entry point against the CPU oracle itself
    return got, want


def _same(got, want):
    for key in ("accept_len", "accept_mask", "next_token"):
        np.testing.assert_array_equal(got[key], want[key])
    np.testing.assert_allclose(np.minimum(got["margins"], 1e30), np.minimum(want["margins"], 1e30),
                               rtol=0, atol=1e-6)


def test_no_alloc_matches_context_entry_point_on_two_calls_in_a_row():
    from paper_2511_13587_b200 import binding as vb
    # first call: relaxed, many images; second call: different sizes and mode, so it runs over
    # whatever the first one left in the shared scratch array
    first = decide_case(901, 16384, 64, 16, 17, 0, MODE_RELAXED, 64, 0.1, 1.0, 0.7)
    second = decide_case(902, 4096 + 40, 5, 8, 8, 0, MODE_STRICT, 1, float("inf"), 0.5, 1.5, off=64)
    for case in (first, second):
        got, want = _both(case, vb)
        _same(got, want)
    got, want = _both(first, vb)                       # and back again
    _same(got, want)


def test_no_alloc_rejects_sizes_beyond_its_fixed_scratch():
    import torch
    from paper_2511_13587_b200 import binding as vb
    z = torch.zeros(64, dtype=torch.float32, device="cuda")
    zi = torch.zeros(64, dtype=torch.int32, device="cuda")
    base = dict(target_probs=z, vocab=8, vocab_offset=0, n_rows_per_seq=2, first_row=0, drafts=zi,
                n_images=1, n_draft_max=1, draft_probs=z, uniforms=z, accept_len=zi, next_token=zi)
    for bad in (dict(n_images=65), dict(n_draft_max=17, n_rows_per_seq=18), dict(vocab=65537),
                dict(mode=MODE_RELAXED, nbr_k=65, nbr_row_ptr=zi, nbr_col=zi)):
        with pytest.raises(vb.VvsError) as e:
            vb.vvs_decide_noalloc(**dict(base, **bad))
        assert e.value.status == -2, bad
    # a candidate tree needs scratch rows the fixed array does not have: refused, not decided as a chain
    for bad in (dict(tree_parent=zi), dict(accept_path=zi)):
        with pytest.raises(vb.VvsError) as e:
            vb.vvs_decide_noalloc(**dict(base, **bad))
        assert e.value.status == -1, bad
