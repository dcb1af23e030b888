"""Policy and codec together: the policy chooses a stored form (level, kept fraction) per entry
from sizes that the codec's own size arithmetic reports; executing the choices on the GPU
(token dropping + encode) must write exactly the bytes the policy budgeted, and every stored
entry must load back as what the oracle decodes from the oracle's encoding of the same form."""
import numpy as np
import pytest
import torch

import oracle
import workloads
from test_gpu_parity import kvh, new_status, to_np16  # noqa: F401

pytestmark = pytest.mark.gpu


def test_policy_choices_executed_on_the_gpu(kvh):
    l, c, n_entries = 2, 1024, 12
    freq, tokens, forms, quality = workloads.policy_entries(n_entries, seed=5)
    tokens = [max(300, n // 16) for n in tokens]                  # short contexts keep the oracle fast
    options, begin, kept_of = [], [0], []
    for i, n in enumerate(tokens):
        for j, (level, keep) in enumerate(forms):
            n_recent = max(0, int(n * keep) - 4)
            runs, n_kept = kvh.keep_sinks_and_recent(n, 4, n_recent)
            options.append((kvh.plan_chunks(l, c, n_kept, level)[1], quality[i][j]))
            kept_of.append((runs, n_kept))
        begin.append(len(options))
    full = sum(options[begin[i]][0] for i in range(n_entries))
    capacity = full // 12
    choice, used, _ = kvh.policy_assign(freq, options, begin, 2.0, 25e9, capacity)
    assert used <= capacity and (choice >= 0).sum() >= 3 and (choice < 0).sum() >= 1

    store = torch.empty(capacity, dtype=torch.uint8, device="cuda")           # the tier
    status = new_status()
    cursor, placed = 0, {}
    for i in range(n_entries):
        if choice[i] < 0:
            continue                                              # evicted: recomputed on a hit
        level, _ = forms[choice[i]]
        runs, n_kept = kept_of[begin[i] + choice[i]]
        size = options[begin[i] + choice[i]][0]
        kv = workloads.make_kv(l, tokens[i], c, seed=900 + i, device="cuda")
        kvh.encode_kept(kv, runs, None, workloads.n_chunks(n_kept), store[cursor:cursor + size], status, level=level)
        want, _ = oracle.encode_kept(to_np16(kv), [(int(r["first"]), int(r["count"])) for r in runs], level)
        assert want.size == size
        assert np.array_equal(store[cursor:cursor + size].cpu().numpy(), want)
        placed[i] = (cursor, size, level, n_kept)
        cursor += size
    assert cursor == used and status.item() == 0                 # the bytes written are the bytes budgeted

    # a hit on every stored entry: one batched load of all of them into a shared pool
    descs, pt_base = [], 0
    for i, (off, size, level, n_kept) in placed.items():
        d, total = kvh.plan_chunks(l, c, n_kept, level, stream_base=off, pt_base=pt_base)
        assert total == size
        descs.append(d)
        pt_base += workloads.n_pages(n_kept) + (-workloads.n_pages(n_kept)) % 16
    descs = np.concatenate(descs)
    table = workloads.shuffled_page_table(pt_base, pt_base, seed=6)
    pool = kvh.Pool.allocate(l, pt_base, c)
    kvh.decode_batch(store, kvh.descs_to_tensor(descs, "cuda"), len(descs), table.cuda(), pool, status)
    assert status.item() == 0
    i, (off, size, level, n_kept) = next(iter(placed.items()))
    vals = np.concatenate([oracle.decode_chunk_values(store[off:off + size].cpu().numpy()[a:], level, l, c, n)
                           for a, n in zip(np.cumsum([0] + [kvh.level_bytes(level, l, c, 256)] * (workloads.n_chunks(n_kept) - 1)),
                                           [256] * (workloads.n_chunks(n_kept) - 1) + [n_kept - 256 * (workloads.n_chunks(n_kept) - 1)])],
                          axis=2)
    pages = table[:workloads.n_pages(n_kept)].long().cuda()
    got = to_np16(pool.tensor[:, :, pages]).reshape(l, 2, -1, c)[:, :, :n_kept]
    assert np.array_equal(got, vals)
