"""CPU oracle for the draft-target matching and prefix-tree packing of Decoupled Speculative Verification.

TEST INFRASTRUCTURE ONLY.  Only the tests, the smoke check and the benchmark's cpu-baseline / reference arm may
import this module; the CUDA library never does, and this module imports nothing from the CUDA path.  Plain Python
over token lists, written from the definitions, not tuned.

What it computes (paper Sec. 3.2, "Draft-target matching process" and "Prefix-tree batching mechanism"):
  * the reference window w = the last n accepted tokens;
  * J(y~) (Eq. 5): every start position at which w occurs in a draft y~;
  * C (Eq. 6): the non-empty suffixes that follow a matched window, over all drafts, as a set;
  * the prefix tree T (Eq. 7): one node per distinct prefix of a member of C; Next(v), child(v, u), pi(v);
  * the packed sequence P: the pending token (the last accepted token) followed by the tree's nodes, with the parent
    row of every node, for the tree-ancestry mask of Fig. 2(c).

Readings where the paper is silent:
  * order and budget of the packing: the paper only bounds the packed length (128 tokens, Sec. 4.3).  Here nodes are
    created level by level (all first tokens, then all second tokens, ..), inside a level in the order of the
    candidates (draft by draft, match position ascending); a node that would exceed the budget is not created and
    the candidates that needed it stop growing.  So every packed tree is a prefix-closed subset of T that keeps all
    shallow nodes, and the rows are in parents-first order;
  * candidates beyond `max_candidates` (in the same order) are ignored;
  * the root row carries the pending token: its K/V is not in the cache yet, so it is the first query row.

Pins (tests/test_dsv_oracle.py): the paper's worked example (Fig. 2(b) as described in the text: the prefix
"tokens" has the next-token set {in, simultaneously, together} and pi(parallel) = "tokens in parallel"); brute-force
equality of the tree's root-to-node paths with the set of all prefixes of C; J against a regular-expression search;
the chain special case |C| = 1; budget and order properties.
"""
from __future__ import annotations

from typing import Dict, List, Sequence, Tuple


def reference_window(accepted: Sequence[int], n: int) -> List[int]:
    """w = y^_{t-n+1:t}: the most recent n accepted tokens (fewer if fewer exist)."""
    return [int(t) for t in accepted[-n:]] if n > 0 else []


def match_positions(draft: Sequence[int], w: Sequence[int]) -> List[int]:
    """J(y~), Eq. 5, as 0-based start positions j with draft[j : j + n] == w."""
    n = len(w)
    if n == 0:
        return []
    return [j for j in range(0, len(draft) - n + 1) if list(draft[j:j + n]) == list(w)]


def candidate_suffixes(drafts: Sequence[Sequence[int]], w: Sequence[int], max_candidates: int = 1 << 30) -> List[List[int]]:
    """C, Eq. 6, in draft order then match order; only suffixes with at least one token (j + n <= |y~| in the
    paper's 1-based positions).  Equal suffixes are kept here (the tree merges them)."""
    n = len(w)
    out: List[List[int]] = []
    for d in drafts:
        for j in match_positions(d, w):
            if j + n < len(d) and len(out) < max_candidates:
                out.append([int(t) for t in d[j + n:]])
    return out


def prefix_tree(cands: Sequence[Sequence[int]], max_nodes: int) -> Tuple[List[int], List[int]]:
    """T, Eq. 7, built level by level under a node budget.  Returns (token of node 1.., parent of node 1..) with node 0
    the root (empty prefix); parents precede children."""
    tok: List[int] = []
    par: List[int] = []
    child: Dict[Tuple[int, int], int] = {}
    cur = [0] * len(cands)            # node each candidate has reached
    alive = [True] * len(cands)
    depth = 0
    while True:
        moved = False
        for c, seq in enumerate(cands):
            if not alive[c] or depth >= len(seq):
                alive[c] = False
                continue
            u = int(seq[depth])
            key = (cur[c], u)
            if key not in child:
                if len(tok) >= max_nodes:
                    alive[c] = False
                    continue
                tok.append(u)
                par.append(cur[c])
                child[key] = len(tok)          # node ids start at 1
            cur[c] = child[key]
            moved = True
        if not moved:
            break
        depth += 1
    return tok, par


def pack(accepted: Sequence[int], drafts: Sequence[Sequence[int]], n: int, max_rows: int, max_candidates: int = 64):
    """The packed sequence P for one decoding step: (q_tokens, parent) with row 0 = the pending token (parent -1)."""
    w = reference_window(accepted, n)
    cands = candidate_suffixes(drafts, w, max_candidates) if len(w) == n else []
    tok, par = prefix_tree(cands, max_rows - 1)
    return [int(accepted[-1])] + tok, [-1] + par


def next_set(tok: Sequence[int], par: Sequence[int], node: int) -> List[int]:
    """Next(v): the tokens of v's children (node ids: 0 = root, i >= 1 = i-th created node)."""
    return sorted(tok[i] for i in range(len(tok)) if par[i] == node)


def path_tokens(tok: Sequence[int], par: Sequence[int], node: int) -> List[int]:
    """pi(v): the tokens from the root to v."""
    out: List[int] = []
    while node > 0:
        out.append(tok[node - 1])
        node = par[node - 1]
    return out[::-1]
