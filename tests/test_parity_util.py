"""The comparison harness itself (CPU): a near-tie is tolerated once and the comparison goes on
with the other side's decision imposed; anything else fails."""
import numpy as np
import pytest

import oracle
from gpu_cases import Case, small_config
from parity_util import check_walk, compare_verify


def _as_device_result(case, orc):
    keys = ("node_next", "node_token", "node_mass", "node_thresh")
    res = {k: np.stack([np.asarray(o[k]) for o in orc]) for k in keys}
    D1 = max(len(o["out_tokens"]) for o in orc) + 8
    res["accept_len"] = np.array([o["accept_len"] for o in orc])
    res["out_tokens"] = np.full((len(orc), D1), -1)
    res["out_nodes"] = np.full((len(orc), D1), -1)
    for b, o in enumerate(orc):
        res["out_tokens"][b, : len(o["out_tokens"])] = o["out_tokens"]
        res["out_nodes"][b, : len(o["out_nodes"])] = o["out_nodes"]
    return res


def _rewalk(res, case):
    for b in range(case.B):
        ln, toks, nodes = oracle.walk(res["node_next"][b], res["node_token"][b], case.tokens[b])
        res["accept_len"][b] = ln
        res["out_tokens"][b] = -1
        res["out_nodes"][b] = -1
        res["out_tokens"][b, : ln + 1] = toks
        res["out_nodes"][b, : ln + 1] = nodes


def _case_with_root_threshold_below_one():
    for seed in range(40, 60):
        case = Case(small_config(batch=1, vocab=200, codebook_size=200, k=6), seed=seed)
        o = case.oracle_verify()[0]
        c = oracle.tree_children(case.parent)[0][0]
        if 0.05 < o["node_thresh"][c] < 0.95:
            return case, c
    raise AssertionError("no suitable case")


def test_identical_results_pass_without_ties():
    case = Case(small_config(batch=2), seed=3)
    orc = case.oracle_verify()
    res = _as_device_result(case, orc)
    stats = compare_verify(res, orc, case.parent, case.u_accept.numpy(), rerun=case.oracle_node)
    assert stats["tie_accept"] == stats["tie_cut"] == stats["tie_resample"] == 0 and not stats["dirty_sequences"]
    check_walk(res, case.tokens, 16, orc, stats["dirty_sequences"], None, stats["patched"])


def test_flipped_decision_inside_the_band_is_one_tie_and_the_rest_is_still_checked():
    case, c = _case_with_root_threshold_below_one()
    thr = case.oracle_verify()[0]["node_thresh"][c]
    case.u_accept[0, c] = float(np.float32(thr - 4e-7))          # the oracle accepts, barely
    case._orc = None
    orc = case.oracle_verify()
    assert orc[0]["node_next"][0] == c
    # the other side rejects this child: its later results follow from that decision
    res = _as_device_result(case, orc)
    nxt, tok, tested = case.oracle_node(0, 0, {c: {"accept": False}})
    res["node_next"][0, 0], res["node_token"][0, 0] = nxt, tok
    for ch in oracle.tree_children(case.parent)[0]:
        res["node_mass"][0, ch], res["node_thresh"][0, ch] = tested[ch][:2] if ch in tested else (-1.0, -1.0)
    _rewalk(res, case)
    stats = compare_verify(res, orc, case.parent, case.u_accept.numpy(), rerun=case.oracle_node)
    assert stats["tie_accept"] == 1 and stats["tie_cut"] == 0 and stats["dirty_sequences"] == {0}
    check_walk(res, case.tokens, 16, orc, stats["dirty_sequences"], None, stats["patched"])
    # a wrong value after the tolerated tie is still found
    later = [ch for ch in oracle.tree_children(case.parent)[0] if ch != c and ch in tested]
    if later:
        res["node_mass"][0, later[0]] += 1e-3
        with pytest.raises(AssertionError):
            compare_verify(res, orc, case.parent, case.u_accept.numpy(), rerun=case.oracle_node)


def test_flipped_decision_outside_the_band_fails():
    case, c = _case_with_root_threshold_below_one()
    thr = case.oracle_verify()[0]["node_thresh"][c]
    case.u_accept[0, c] = float(np.float32(thr - 1e-3))
    case._orc = None
    orc = case.oracle_verify()
    res = _as_device_result(case, orc)
    nxt, tok, _ = case.oracle_node(0, 0, {c: {"accept": False}})
    res["node_next"][0, 0], res["node_token"][0, 0] = nxt, tok
    with pytest.raises(AssertionError):
        compare_verify(res, orc, case.parent, case.u_accept.numpy(), rerun=case.oracle_node)
