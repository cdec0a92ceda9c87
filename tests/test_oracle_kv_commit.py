"""Pin for the KV commit (not in the paper; the step that closes the loop of Sec. 3.2): when
every cache row is a function of (token, position), a cache maintained by draft -> accept ->
commit must equal, row for row, the cache plain token-by-token decoding would have written."""
import numpy as np

import oracle


def toy_next(prefix, vocab):
    return (int(prefix[-2]) * 7 + int(prefix[-1]) * 3 + 1) % vocab


def enc(token, pos, H, D, which):
    """Row content a model would have written for `token` at absolute position `pos`."""
    h = np.arange(H)[:, None]
    d = np.arange(D)[None, :]
    return ((token * 131 + pos * 17 + h * 5 + d + which * 3) % 65521).astype(np.uint16)


def test_commit_reproduces_the_cache_of_plain_decoding():
    vocab, m, N, H, D, Lcap = 11, 6, 24, 2, 128, 260
    rng = np.random.default_rng(0)
    T = [3, 5]
    for _ in range(6000):
        T.append(toy_next(T, vocab) if rng.random() < 0.85 else int(rng.integers(0, vocab)))
    T = np.array(T, np.int32)
    sa = oracle.suffix_array(T)
    seq = [1, 4, 2, 8]
    k = np.zeros((1, H, Lcap, D), np.uint16)
    v = np.zeros((1, H, Lcap, D), np.uint16)
    for p, x in enumerate(seq):
        k[0, :, p], v[0, :, p] = enc(x, p, H, D, 0), enc(x, p, H, D, 1)
    moved = 0
    while len(seq) < 200:
        L = len(seq)
        d = oracle.draft(T, sa, vocab, np.array([seq], np.int32), [L], m=m, N=N)
        tok, par, dep, nn = d["tokens"], d["parents"], d["depth"], d["n_nodes"]
        ver = np.zeros((1, N + 1), np.int32)
        ver[0, 0] = toy_next(seq, vocab)
        for i in range(int(nn[0])):
            path, j = [], i
            while j >= 0:
                path.append(int(tok[0, j]))
                j = int(par[0, j])
            ver[0, i + 1] = toy_next(seq + path[::-1], vocab)
            # the model writes the K/V of draft node i at tree slot L + i, position L + depth - 1
            k[0, :, L + i] = enc(int(tok[0, i]), L + int(dep[0, i]) - 1, H, D, 0)
            v[0, :, L + i] = enc(int(tok[0, i]), L + int(dep[0, i]) - 1, H, D, 1)
        al, an, ot = oracle.accept(tok, par, nn, ver, m)
        k, v, new_len = oracle.kv_commit(k, v, np.array([L], np.int32), an, al)
        a = int(al[0])
        assert int(new_len[0]) == L + a
        moved += int((an[0, :a] != np.arange(a)).sum())
        seq += ot[0, :a + 1].tolist()
        # the token produced at the stop gets its row from the model's next forward pass
        p = len(seq) - 1
        k[0, :, p], v[0, :, p] = enc(seq[p], p, H, D, 0), enc(seq[p], p, H, D, 1)
    plain = [1, 4, 2, 8]
    while len(plain) < len(seq):
        plain.append(toy_next(plain, vocab))
    assert seq == plain
    assert moved > 10                     # rows really had to move, not only stay in place
    for p, x in enumerate(plain):
        assert np.array_equal(k[0, :, p], enc(x, p, H, D, 0)), p
        assert np.array_equal(v[0, :, p], enc(x, p, H, D, 1)), p


def test_overlapping_source_and_destination_slots():
    # nodes (1, 3, 4), len 3: slot L+1 is the source of i=0 and the destination of i=1
    H, D, L = 1, 128, 5
    k = (np.arange(12, dtype=np.uint16)[None, None, :, None] * np.ones((1, H, 12, D), np.uint16)).copy()
    v = (k + 100).astype(np.uint16)
    nodes = np.array([[1, 3, 4, -1]], np.int32)
    k2, v2, nl = oracle.kv_commit(k, v, np.array([L], np.int32), nodes, np.array([3], np.int32))
    assert k2[0, 0, :, 0].tolist() == [0, 1, 2, 3, 4, 6, 8, 9, 8, 9, 10, 11]
    assert v2[0, 0, :, 0].tolist() == [100, 101, 102, 103, 104, 106, 108, 109, 108, 109, 110, 111]
    assert nl.tolist() == [8]
