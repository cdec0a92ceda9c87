"""Pins for draft acceptance (Sec. 3.2 "Draft acceptance"): decoding with drafts must
reproduce plain one-token-at-a-time decoding exactly, whatever the drafts were."""
import numpy as np

import oracle


def toy_next(prefix, vocab, noise_key=0):
    """Deterministic stand-in for the verifier: next token from the last two tokens."""
    a, b = int(prefix[-2]), int(prefix[-1])
    return (a * 7 + b * 3 + 1 + noise_key) % vocab


def test_lossless_against_token_by_token_decoding():
    vocab, m, N = 11, 6, 24
    rng = np.random.default_rng(0)
    # datastore: mostly follows the toy rule, with random deviations, so drafts are often
    # right for a few tokens and then wrong
    T = [3, 5]
    for _ in range(6000):
        T.append(toy_next(T, vocab) if rng.random() < 0.85 else int(rng.integers(0, vocab)))
    T = np.array(T, np.int32)
    sa = oracle.suffix_array(T)
    prompt = [1, 4, 2, 8]
    plain = list(prompt)
    while len(plain) < 200:
        plain.append(toy_next(plain, vocab))

    seq = list(prompt)
    steps = 0
    accepted_total = 0
    while len(seq) < 200:
        ctx = np.array(seq, np.int32)
        d = oracle.draft(T, sa, vocab, ctx[None], [len(seq)], m=m, N=N)
        tok, par, nn = d["tokens"], d["parents"], d["n_nodes"]
        ver = np.zeros((1, N + 1), np.int32)
        ver[0, 0] = toy_next(seq, vocab)
        for i in range(int(nn[0])):
            path, j = [], i
            while j >= 0:
                path.append(int(tok[0, j]))
                j = int(par[0, j])
            ver[0, i + 1] = toy_next(seq + path[::-1], vocab)
        al, an, ot = oracle.accept(tok, par, nn, ver, max_depth=m)
        new = ot[0, :al[0] + 1].tolist()
        assert all(t >= 0 for t in new)
        # accepted nodes form a root-to-node path
        prev = -1
        for dpt in range(al[0]):
            node = an[0, dpt]
            assert par[0, node] == prev and d["depth"][0, node] == dpt + 1
            prev = node
        seq += new
        accepted_total += int(al[0])
        steps += 1
    assert seq[:200] == plain[:200]
    assert accepted_total / steps > 0.5        # drafts were actually used


def test_accept_edge_cases():
    # empty tree -> nothing accepted, the verifier's first token is returned
    tok = np.full((1, 4), -1, np.int32)
    par = np.full((1, 4), -1, np.int32)
    al, an, ot = oracle.accept(tok, par, [0], np.array([[7, 1, 2, 3, 4]], np.int32), 3)
    assert al.tolist() == [0] and ot[0].tolist() == [7, -1, -1, -1] and (an == -1).all()
    # padding slots (token -1) are never matched even if the verifier says -1
    al, an, ot = oracle.accept(tok, par, [0], np.array([[-1, 1, 2, 3, 4]], np.int32), 3)
    assert al.tolist() == [0]
    # chain accepted to the depth limit
    tok = np.array([[5, 6, 7, 8]], np.int32)
    par = np.array([[-1, 0, 1, 2]], np.int32)
    ver = np.array([[5, 6, 7, 8, 9]], np.int32)
    al, an, ot = oracle.accept(tok, par, [4], ver, 4)
    assert al.tolist() == [4] and an[0].tolist() == [0, 1, 2, 3] and ot[0].tolist() == [5, 6, 7, 8, 9]
    al, an, ot = oracle.accept(tok, par, [4], ver, 2)        # depth limit stops the walk
    assert al.tolist() == [2] and ot[0].tolist() == [5, 6, 7]
    # same token under different parents: only the child of the current node counts
    tok = np.array([[1, 2, 9, 9]], np.int32)
    par = np.array([[-1, -1, 0, 1]], np.int32)
    ver = np.array([[2, 0, 9, 3, 4]], np.int32)
    al, an, ot = oracle.accept(tok, par, [4], ver, 3)
    assert al.tolist() == [2] and an[0, :2].tolist() == [1, 3] and ot[0, :3].tolist() == [2, 9, 4]
