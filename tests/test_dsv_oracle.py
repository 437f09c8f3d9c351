"""Pins of the matching / prefix-tree oracle (Sec. 3.2, Eq. 5-7) against what the paper and the definitions fix."""
import os
import re

import numpy as np

from oracle import dsv_oracle as D

GOLD = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "paper_dsv_example.txt")


def test_papers_worked_example():
    cands, checks = [], []
    for line in open(GOLD):
        line = line.strip()
        if line.startswith("candidate ="):
            cands.append(line.split("=", 1)[1].split())
        elif "->" in line and not line.startswith("#"):
            k, v = line.split("=", 1)
            checks.append((k.strip(), v.split("->")[0].split(), v.split("->")[1].split()))
    vocab = {}
    ids = [[vocab.setdefault(wd, len(vocab)) for wd in c] for c in cands]
    word = {i: wd for wd, i in vocab.items()}
    tok, par = D.prefix_tree(ids, 100)
    assert len(tok) == 5                                     # tokens, in, simultaneously, together, parallel
    node_of = {tuple(D.path_tokens(tok, par, v)): v for v in range(1, len(tok) + 1)}
    for kind, key, want in checks:
        if kind == "next_of_prefix":
            v = node_of[tuple(vocab[wd] for wd in key)]
            assert sorted(word[t] for t in D.next_set(tok, par, v)) == sorted(want)
        else:
            v = [i for i in range(1, len(tok) + 1) if word[tok[i - 1]] == key[0]][0]
            assert [word[t] for t in D.path_tokens(tok, par, v)] == want
    assert D.next_set(tok, par, 0) == [vocab["tokens"]]      # the root has the single shared first token


def test_match_positions_equal_a_regular_expression_search():
    rng = np.random.default_rng(5)
    for _ in range(200):
        n = int(rng.integers(1, 4))
        draft = rng.integers(0, 3, size=int(rng.integers(0, 30))).tolist()
        w = rng.integers(0, 3, size=n).tolist()
        text, pat = "".join(map(str, draft)), "".join(map(str, w))
        want = [m.start() for m in re.finditer(f"(?={pat})", text)]    # overlapping occurrences
        assert D.match_positions(draft, w) == want


def test_tree_paths_are_exactly_the_prefixes_of_the_candidates():
    rng = np.random.default_rng(9)
    for _ in range(100):
        n = 2
        drafts = [rng.integers(0, 4, size=int(rng.integers(3, 25))).tolist() for _ in range(int(rng.integers(1, 4)))]
        acc = rng.integers(0, 4, size=5).tolist()
        w = D.reference_window(acc, n)
        cands = D.candidate_suffixes(drafts, w)
        # Eq. 6 by brute force over every (draft, position)
        brute = [d[j + n:] for d in drafts for j in range(len(d) - n + 1) if d[j:j + n] == w and j + n < len(d)]
        assert cands == brute
        tok, par = D.prefix_tree(cands, 10_000)
        paths = {tuple(D.path_tokens(tok, par, v)) for v in range(1, len(tok) + 1)}
        prefixes = {tuple(c[:k]) for c in cands for k in range(1, len(c) + 1)}
        assert paths == prefixes and len(paths) == len(tok)              # one node per distinct prefix
        assert all(0 <= par[i] <= i for i in range(len(tok)))            # parents first (node ids are 1-based)
        for v in range(0, len(tok) + 1):                                 # Next(v) by its definition
            pv = tuple(D.path_tokens(tok, par, v))
            want = sorted({c[len(pv)] for c in cands if tuple(c[:len(pv)]) == pv and len(c) > len(pv)})
            assert D.next_set(tok, par, v) == want


def test_single_candidate_is_a_chain_and_no_match_is_the_bare_root():
    q, p = D.pack([7, 1, 2, 3], [[9, 1, 2, 3, 4, 5, 6]], 3, 128)
    assert q == [3, 4, 5, 6] and p == [-1, 0, 1, 2]
    q, p = D.pack([7, 1, 2, 3], [[9, 1, 2, 4, 4, 5, 6]], 3, 128)
    assert q == [3] and p == [-1]
    q, p = D.pack([7, 1, 2, 3], [[9, 1, 2, 3]], 3, 128)                  # match at the very end: empty suffix, dropped
    assert q == [3] and p == [-1]
    q, p = D.pack([2, 3], [[1, 2, 3, 4]], 3, 128)                        # fewer accepted tokens than the window
    assert q == [3] and p == [-1]


def test_budget_keeps_shallow_nodes_and_candidate_order():
    cands = [[1, 2, 3, 4, 5], [1, 2, 9, 9], [6, 7, 8]]
    tok, par = D.prefix_tree(cands, 100)
    assert tok == [1, 6, 2, 7, 3, 9, 8, 4, 9, 5] and par == [0, 0, 1, 2, 3, 3, 4, 5, 6, 8]
    tok, par = D.prefix_tree(cands, 5)                                   # level order: depth 1, depth 2, then one of depth 3
    assert tok == [1, 6, 2, 7, 3] and par == [0, 0, 1, 2, 3]
    full = {tuple(D.path_tokens(*D.prefix_tree(cands, 100), v)) for v in range(1, 11)}
    cut = {tuple(D.path_tokens(tok, par, v)) for v in range(1, 6)}
    assert cut <= full and all(len(p) <= 3 for p in cut)
    # candidate cap: later matches are ignored
    assert D.candidate_suffixes([[1, 5, 1, 6, 1, 7]], [1], max_candidates=2) == [[5, 1, 6, 1, 7], [6, 1, 7]]
