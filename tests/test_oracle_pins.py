"""Pins of the fp64 oracle against things other than itself (CPU only).

Each test checks the oracle against a closed form, a library routine, a hand-derived table
or brute force written differently, so that a dropped term, a wrong sign or index, or a
transposed operand in ``oracle/aspd_oracle.c`` fails at least one of them.
"""
import math
import os

import numpy as np
import pytest
import torch

import oracle
from oracle.run import run_workload
from paper_2508_08895_b200 import workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "worked_example.txt")


def load_example():
    rows = []
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        idx, br, st, pos, vis = line.split()
        rows.append((int(idx), int(br), int(st), int(pos), [int(x) for x in vis.split(",")]))
    return rows


# --------------------------------------------------------------------------- Eq. 2-4
def test_worked_example_positions_and_mask():
    rows = load_example()
    branch = [r[1] for r in rows]
    stage = [r[2] for r in rows]
    pos = oracle.dense_positions(branch, stage)
    assert pos.tolist() == [r[3] for r in rows]
    vis = oracle.dense_visible(branch, stage)
    for i, r in enumerate(rows):
        assert np.flatnonzero(vis[i]).tolist() == r[4], i


def test_main_branch_position_is_flat_index_and_stage_order():
    """Eq. 4: a main token's position is its index in the complete sequence; every position
    issued in a stage exceeds every position issued before that stage (so Eq. 3's
    different-stage case can never expose a later token)."""
    rng = np.random.default_rng(5)
    for _ in range(50):
        branch, stage = [], []
        st = 0
        for _seg in range(rng.integers(1, 4)):
            for _ in range(rng.integers(1, 5)):
                branch.append(-1); stage.append(st)
            st += 1
            nb = int(rng.integers(1, 4))
            lens = rng.integers(1, 5, size=nb)
            for step in range(int(lens.max())):
                for b in range(nb):
                    if step < lens[b]:
                        branch.append(b); stage.append(st)
            st += 1
        branch.append(-1); stage.append(st)
        pos = oracle.dense_positions(branch, stage)
        branch, stage = np.array(branch), np.array(stage)
        assert (pos[branch < 0] == np.flatnonzero(branch < 0)).all()
        for s in range(1, st + 1):
            assert pos[stage == s].min() > pos[stage < s].max() or pos[stage == s].min() == np.flatnonzero(stage == s)[0]
            assert pos[stage == s].min() == np.flatnonzero(stage == s)[0]
        # same timestep => same position for every branch of a stage (shared position IDs)
        for s in np.unique(stage[branch >= 0]):
            start = np.flatnonzero(stage == s)[0]
            for b in np.unique(branch[stage == s]):
                mine = pos[(stage == s) & (branch == b)]
                assert mine.tolist() == list(range(start, start + len(mine)))


def test_descriptor_positions_closed_form():
    """Parallel token k of a branch -> P + k; first serial token after the segment ->
    P + sum of branch lengths (its index in the complete sequence)."""
    wl = W.build_segment_workload("t", 1, 2, 1, 8, "f32", 100.0, [5], [[2, 0, 1]], [[1, 1, 1]], serial_steps=2)
    par = [p for p in wl.phases if p.label == "parallel-step"][0]
    pos, slot, req = oracle.new_tokens(par.desc, oracle.MODE_BRANCH)
    assert pos.tolist() == [5 + 2, 5 + 0, 5 + 1]
    assert slot.tolist() == [16 + 2, 32 + 0, 48 + 1]      # page-aligned branch regions after the 5-token prefix
    ser = [p for p in wl.phases if p.label.startswith("serial")]
    p0, s0, _ = oracle.new_tokens(ser[0].desc, oracle.MODE_SERIAL)
    p1, s1, _ = oracle.new_tokens(ser[1].desc, oracle.MODE_SERIAL)
    assert p0.tolist() == [5 + 3 + 1 + 2] and p1.tolist() == [5 + 3 + 1 + 2 + 1]
    assert s0.tolist() == [64] and s1.tolist() == [65]


def test_descriptor_matches_worked_example():
    """The descriptor form reproduces the hand-derived table's first parallel stage and the
    serial token after it (positions and visible sets, as integers)."""
    rows = load_example()
    # final state of stage 1: P = 5, branches of 3, 1, 2 tokens; the last decoding step has
    # only branch 0 alive (flat index 10)
    wl = W.build_segment_workload("t", 1, 2, 1, 8, "f32", 100.0, [5], [[2, 1, 2]], [[1, 0, 0]], serial_steps=1)
    par = [p for p in wl.phases if p.label == "parallel-step"][0]
    pos, slot, _ = oracle.new_tokens(par.desc, oracle.MODE_BRANCH)
    assert pos.tolist() == [rows[10][3]]
    n_slots = int(par.desc["n_pages"][0]) * wl.page_size
    vis = oracle.visible_slots(par.desc, oracle.MODE_BRANCH, n_slots)
    # map flat indices of the table to slots: prefix i -> i; branch b token k -> br_off[b] + k
    off = par.desc["br_kv_off"]
    flat_to_slot = {i: i for i in range(5)}
    flat_to_slot.update({5: off[0], 8: off[0] + 1, 10: off[0] + 2, 6: off[1], 7: off[2], 9: off[2] + 1})
    assert sorted(np.flatnonzero(vis[0]).tolist()) == sorted(int(flat_to_slot[j]) for j in rows[10][4])
    ser = [p for p in wl.phases if p.label == "serial-0"][0]
    pos, slot, _ = oracle.new_tokens(ser.desc, oracle.MODE_SERIAL)
    assert pos.tolist() == [rows[11][3]]
    flat_to_slot[11] = int(ser.desc["tail_off"][0])
    vis = oracle.visible_slots(ser.desc, oracle.MODE_SERIAL, n_slots)
    assert sorted(np.flatnonzero(vis[0]).tolist()) == sorted(int(flat_to_slot[j]) for j in rows[11][4])


# ------------------------------------------------------------------------------ RoPE
def test_rope_closed_forms():
    rng = np.random.default_rng(0)
    # d = 2: a plane rotation by pos radians, whatever theta is
    for pos, theta in [(0.0, 10000.0), (1.0, 10000.0), (3.0, 7.0), (1000.0, 1e6)]:
        x = rng.standard_normal(2)
        y = oracle.rope(x, pos, theta)
        c, s = math.cos(pos), math.sin(pos)
        np.testing.assert_allclose(y, [x[0] * c - x[1] * s, x[1] * c + x[0] * s], atol=1e-12)
    # pos = 0: identity; any pos: norm preserved; complex-multiplication form
    for d, theta in [(8, 10000.0), (64, 10000.0), (128, 1e6)]:
        x = rng.standard_normal(d)
        np.testing.assert_array_equal(oracle.rope(x, 0.0, theta), x)
        for pos in [1.0, 17.0, 16640.0]:
            y = oracle.rope(x, pos, theta)
            assert abs(np.linalg.norm(y) - np.linalg.norm(x)) < 1e-10
            z = (x[: d // 2] + 1j * x[d // 2:]) * np.exp(1j * pos * theta ** (-np.arange(d // 2) * 2.0 / d))
            np.testing.assert_allclose(y, np.concatenate([z.real, z.imag]), atol=1e-10)


def test_rope_rotations_compose():
    """RoPE(RoPE(x, p), delta) = RoPE(x, p + delta): what re-rotating cached keys relies on."""
    rng = np.random.default_rng(4)
    x = rng.standard_normal(128)
    for p, dlt in [(5.0, 11.0), (1040.0, -17.0), (16384.0, 300.0)]:
        np.testing.assert_allclose(oracle.rope(oracle.rope(x, p, 1e6), dlt, 1e6), oracle.rope(x, p + dlt, 1e6), atol=1e-9)


def _library_rotary(x, positions, theta):
    """cos/sin tables from the definition of the frequencies, applied by the rotate-half
    routine of the `transformers` Llama implementation (a library routine)."""
    llama = pytest.importorskip("transformers.models.llama.modeling_llama")
    x = torch.as_tensor(np.asarray(x, dtype=np.float64))          # [T][H][d]
    d = x.shape[-1]
    inv = 1.0 / (theta ** (torch.arange(0, d, 2, dtype=torch.float64) / d))
    ang = torch.as_tensor(np.asarray(positions, dtype=np.float64))[:, None] * inv[None, :]
    emb = torch.cat([ang, ang], dim=-1)
    fn = getattr(llama.apply_rotary_pos_emb, "__wrapped__", llama.apply_rotary_pos_emb)
    out, _ = fn(x[None], x[None], emb.cos()[None], emb.sin()[None], unsqueeze_dim=2)
    return out[0].numpy()


def test_rope_matches_library_rotary():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((5, 3, 64))
    positions = [0, 1, 7, 300, 16640]
    ref = _library_rotary(x, positions, 10000.0)
    for t, p in enumerate(positions):
        for h in range(3):
            np.testing.assert_allclose(oracle.rope(x[t, h], float(p), 10000.0), ref[t, h], atol=1e-9)


def test_global_position_shift_leaves_attention_unchanged():
    """RoPE scores depend on position differences only: prepending c dummy-invisible offset
    is emulated by comparing a standalone causal sequence at positions 0.. with the same
    sequence at positions 1000.. through the library attention."""
    rng = np.random.default_rng(2)
    T, H, d = 9, 2, 16
    q, k, v = (rng.standard_normal((T, H, d)) for _ in range(3))
    outs = []
    for c in (0, 1000):
        pos = np.arange(T) + c
        qh = np.stack([[oracle.rope(q[t, h], float(pos[t]), 100.0) for h in range(H)] for t in range(T)])
        kh = np.stack([[oracle.rope(k[t, h], float(pos[t]), 100.0) for h in range(H)] for t in range(T)])
        o = torch.nn.functional.scaled_dot_product_attention(
            torch.tensor(qh).permute(1, 0, 2)[None], torch.tensor(kh).permute(1, 0, 2)[None],
            torch.tensor(v).permute(1, 0, 2)[None], is_causal=True)
        outs.append(o.numpy())
    np.testing.assert_allclose(outs[0], outs[1], atol=1e-9)


# ------------------------------------------------------------- Eq. 1 on tiny inputs
def test_dense_attention_equals_bruteforce_masked_softmax():
    """Eq. 1 written out with an additive 0 / -inf matrix built from the hand-derived table."""
    rows = load_example()
    L, Hq, Hkv, d, theta, scale = len(rows), 4, 2, 8, 50.0, 0.4
    rng = np.random.default_rng(3)
    q = rng.standard_normal((L, Hq, d)); k = rng.standard_normal((L, Hkv, d)); v = rng.standard_normal((L, Hkv, d))
    out = oracle.dense_attn(q, k, v, [r[1] for r in rows], [r[2] for r in rows], theta, scale)
    pos = [r[3] for r in rows]
    M = np.full((L, L), -np.inf)
    for i, r in enumerate(rows):
        for j in r[4]:
            M[i, j] = 0.0
    qh = _library_rotary(q, pos, theta)
    kh = _library_rotary(k, pos, theta)
    for h in range(Hq):
        logits = (qh[:, h, :] @ kh[:, h // (Hq // Hkv), :].T) * scale + M
        p = np.exp(logits - logits.max(axis=1, keepdims=True))
        p /= p.sum(axis=1, keepdims=True)
        np.testing.assert_allclose(out[:, h, :], p @ v[:, h // (Hq // Hkv), :], atol=1e-12)


def _sdpa_causal_last(q_last, k_seq, v_seq, positions, theta, scale, G):
    """Textbook causal attention (library SDPA, fp64) over a standalone sequence; returns the
    last token's output [Hq][d].  q is only needed for the last token."""
    T, Hkv, d = k_seq.shape
    kh = torch.tensor(_library_rotary(k_seq, positions, theta)).permute(1, 0, 2)       # [Hkv][T][d]
    qh = torch.tensor(_library_rotary(q_last[None], positions[-1:], theta))[0]          # [Hq][d]
    Hq = qh.shape[0]
    qfull = torch.zeros(Hq, T, d, dtype=torch.float64)
    qfull[:, -1, :] = qh
    kk = kh.repeat_interleave(G, dim=0)
    vv = torch.tensor(np.asarray(v_seq, dtype=np.float64)).permute(1, 0, 2).repeat_interleave(G, dim=0)
    o = torch.nn.functional.scaled_dot_product_attention(qfull[None], kk[None], vv[None], is_causal=True, scale=scale)
    return o[0, :, -1, :].numpy()


def _branch_tokens(wl, r=0):
    """Raw K/V of prefix and of each branch (prior + new) of request 0, from the phases."""
    ph = {p.label: p for p in wl.phases}
    P = int(ph["parallel-step"].desc["prefix_len"][r])
    kpre, vpre = ph["fill-prefix"].k_new[:P], ph["fill-prefix"].v_new[:P]
    d = ph["parallel-step"].desc
    nb = int(d["n_branches"][r])
    prior = (d["br_kv_len"] - d["br_q_len"])[:nb]
    qn = d["br_q_len"][:nb]
    kb, vb, at, at_new = [], [], 0, 0
    for b in range(nb):
        kp = ph["fill-branches"].k_new[at:at + prior[b]] if "fill-branches" in ph else np.zeros((0,) + kpre.shape[1:])
        vp = ph["fill-branches"].v_new[at:at + prior[b]] if "fill-branches" in ph else np.zeros((0,) + kpre.shape[1:])
        kn = ph["parallel-step"].k_new[at_new:at_new + qn[b]]
        vn = ph["parallel-step"].v_new[at_new:at_new + qn[b]]
        kb.append(np.concatenate([kp, kn])); vb.append(np.concatenate([vp, vn]))
        at += prior[b]; at_new += qn[b]
    return P, kpre, vpre, kb, vb, qn


def test_each_branch_equals_standalone_causal_sequence():
    """From a branch's point of view decoding is ordinary causal decoding of prefix + branch
    with positions 0 .. P + len - 1 (Section 3.2, 'The Parallel Branch's Perspective')."""
    wl = W.config_tiny()
    run = run_workload(wl)
    out = run.outputs[0]
    P, kpre, vpre, kb, vb, qn = _branch_tokens(wl)
    qs = [p for p in wl.phases if p.label == "parallel-step"][0].q
    for b in range(len(kb)):
        kseq = np.concatenate([kpre, kb[b]]); vseq = np.concatenate([vpre, vb[b]])
        ref = _sdpa_causal_last(qs[b], kseq, vseq, np.arange(len(kseq)), wl.theta, wl.sm_scale, wl.G)
        np.testing.assert_allclose(out[b], ref, atol=1e-10)


def test_single_branch_equals_ordinary_causal_decode():
    """N = 1: the parallel step is plain causal decode (library SDPA) and equals the serial path."""
    wl = W.build_segment_workload("n1", 9, 4, 2, 16, "f32", 10000.0, [37], [[5]], [[1]])
    run = run_workload(wl)
    P, kpre, vpre, kb, vb, _ = _branch_tokens(wl)
    q = wl.phases[-1].q
    kseq = np.concatenate([kpre, kb[0]]); vseq = np.concatenate([vpre, vb[0]])
    ref = _sdpa_causal_last(q[0], kseq, vseq, np.arange(len(kseq)), wl.theta, wl.sm_scale, wl.G)
    np.testing.assert_allclose(run.outputs[0][0], ref, atol=1e-10)
    # the same tokens as one serial sequence: prefix of 37 + 5 tokens, 6th decoded serially
    ws = W.build_segment_workload("n1s", 9, 4, 2, 16, "f32", 10000.0, [42], [[]], [[]], serial_steps=1)
    rs = oracle.run.OracleRun(ws)
    fill = ws.phases[0]
    fill.k_new[:] = kseq[:42]; fill.v_new[:] = vseq[:42]
    rs.step(fill)
    ser = ws.phases[1]
    ser.k_new[:] = kseq[42:]; ser.v_new[:] = vseq[42:]; ser.q[:] = q
    o = rs.step(ser)
    np.testing.assert_allclose(o[0], ref, atol=1e-10)


def test_branch_permutation_permutes_outputs():
    prior, newq = [7, 3, 12], [1, 1, 1]
    wl = W.build_segment_workload("p", 4, 4, 2, 16, "f32", 10000.0, [21], [prior], [newq])
    base = run_workload(wl).outputs[0]
    P, kpre, vpre, kb, vb, _ = _branch_tokens(wl)
    q = wl.phases[-1].q
    perm = [2, 0, 1]
    wp = W.build_segment_workload("p2", 4, 4, 2, 16, "f32", 10000.0, [21], [[prior[i] for i in perm]], [newq])
    ph = {p.label: p for p in wp.phases}
    ph["fill-prefix"].k_new[:] = kpre; ph["fill-prefix"].v_new[:] = vpre
    ph["fill-branches"].k_new[:] = np.concatenate([kb[i][:-1] for i in perm])
    ph["fill-branches"].v_new[:] = np.concatenate([vb[i][:-1] for i in perm])
    ph["parallel-step"].k_new[:] = np.stack([kb[i][-1] for i in perm])
    ph["parallel-step"].v_new[:] = np.stack([vb[i][-1] for i in perm])
    ph["parallel-step"].q[:] = q[perm]
    outp = run_workload(wp).outputs[0]
    np.testing.assert_array_equal(outp, base[perm])


@pytest.mark.parametrize("mask", [oracle.MASK_BRANCH_INVISIBLE, oracle.MASK_SHARED])
def test_dense_and_descriptor_forms_agree(mask):
    """oracle-S (engine prose) computes exactly what oracle-D (Eq. 1-4) does, whatever the
    arrangement of tokens in memory: branch-contiguous slots vs interleaved decoding order.
    Also under the ablation's visible mask."""
    rng = np.random.default_rng(11)
    for trial in range(12):
        P = int(rng.integers(1, 9)); nb = int(rng.integers(1, 5))
        lens = [int(x) for x in rng.integers(1, 6, size=nb)]
        n_serial = int(rng.integers(1, 3))
        # one decode step at a time through the descriptor oracle
        Hq, Hkv, d, theta = 4, 2, 8, 100.0
        flat_branch, flat_stage, flat_q, flat_k, flat_v, outs = [], [], [], [], [], []
        prefix_wl = W.build_segment_workload("f", 100 + trial, Hq, Hkv, d, "f32", theta, [P], [[0] * nb], [[0] * nb])
        # prefix as main-branch tokens
        fill = prefix_wl.phases[0]
        for t in range(P):
            flat_branch.append(-1); flat_stage.append(0)
            flat_k.append(fill.k_new[t]); flat_v.append(fill.v_new[t]); flat_q.append(np.zeros((Hq, d)))
        # reference layout: final lengths known, decode step by step
        final = W.build_segment_workload("g", 100 + trial, Hq, Hkv, d, "f32", theta, [P], [[0] * nb], [lens],
                                         serial_steps=n_serial)
        run = oracle.run.OracleRun(final, mask)
        run.step(final.phases[0])                               # prefix
        par = [p for p in final.phases if p.label == "parallel-step"][0]
        # split the one-shot parallel phase (q_len = len) into per-token steps
        starts = np.concatenate([[0], np.cumsum(lens)])
        step_out = {}
        for step in range(max(lens)):
            live = [b for b in range(nb) if step < lens[b]]
            desc = {k: v.copy() for k, v in par.desc.items()}
            desc["br_kv_len"] = np.array([min(step + 1, lens[b]) for b in range(nb)], dtype=np.int32)
            desc["br_q_len"] = np.array([1 if b in live else 0 for b in range(nb)], dtype=np.int32)
            idx = [int(starts[b] + step) for b in live]
            ph = W.Phase(W.MODE_BRANCH, desc, par.k_new[idx], par.v_new[idx], par.q[idx], True)
            o = run.step(ph)
            for n, b in enumerate(live):
                flat_branch.append(b); flat_stage.append(1)
                flat_k.append(par.k_new[idx[n]]); flat_v.append(par.v_new[idx[n]]); flat_q.append(par.q[idx[n]])
                outs.append(o[n])
        for ph in [p for p in final.phases if p.label.startswith("serial")]:
            o = run.step(ph)
            flat_branch.append(-1); flat_stage.append(2)
            flat_k.append(ph.k_new[0]); flat_v.append(ph.v_new[0]); flat_q.append(ph.q[0]); outs.append(o[0])
        dense = oracle.dense_attn(np.array(flat_q), np.array(flat_k), np.array(flat_v), flat_branch, flat_stage,
                                  theta, final.sm_scale, mask=mask)
        np.testing.assert_allclose(dense[P:], np.array(outs), atol=1e-12)


@pytest.mark.parametrize("mask", [oracle.MASK_BRANCH_INVISIBLE, oracle.MASK_SHARED])
def test_whole_branches_at_once_equal_dense_form(mask):
    """Teacher-forcing layout: every branch gets all its tokens in one step (block-diagonal mask
    across branches, causal inside a branch).  The descriptor form equals Eq. 1-4 taken literally
    for every one of those tokens, whatever order the branches are laid out in."""
    Hq, Hkv, d, theta = 4, 2, 16, 1e4
    P, lens = 6, [4, 1, 7]
    wl = W.build_segment_workload("tf", 23, Hq, Hkv, d, "f32", theta, [P], [[0, 0, 0]], [lens], serial_steps=1)
    run = run_workload(wl, mask)
    fill = wl.phases[0]
    par = [p for p in wl.phases if p.label == "parallel-step"][0]
    ser = wl.phases[-1]
    # flat list in training order: prefix, then the branches one after the other, then the serial token
    branch = [-1] * P + [b for b, n in enumerate(lens) for _ in range(n)] + [-1]
    stage = [0] * P + [1] * sum(lens) + [2]
    q = np.concatenate([np.zeros((P, Hq, d)), par.q, ser.q])
    k = np.concatenate([fill.k_new, par.k_new, ser.k_new])
    v = np.concatenate([fill.v_new, par.v_new, ser.v_new])
    dense = oracle.dense_attn(q, k, v, branch, stage, theta, wl.sm_scale, mask=mask)
    np.testing.assert_allclose(run.outputs[0], dense[P:P + sum(lens)], atol=1e-12)
    np.testing.assert_allclose(run.outputs[1][0], dense[-1], atol=1e-12)
    pos, _, _ = oracle.new_tokens(par.desc, oracle.MODE_BRANCH)
    assert pos.tolist() == [P + i for n in lens for i in range(n)]


def test_second_parallel_stage_descriptor_form_equals_dense_form():
    """A request that opens a second parallel stage (regions of the first stage and the serial
    tokens between the stages marked as shared): the descriptor form gives the positions and
    visible sets of the hand-derived table, and the same outputs as Eq. 1-4 taken literally."""
    rows = load_example()
    Hq, Hkv, d, theta = 4, 2, 16, 1e4
    wl = W.build_two_stage_workload("ts", 5, Hq, Hkv, d, "f32", theta, 5, [3, 1, 2], 2, [1, 0], [1, 1], serial_steps=1)
    run = run_workload(wl)
    # raw values by logical slot
    n_slots = int(wl.phases[0].desc["n_pages"][0]) * wl.page_size
    kk = np.zeros((n_slots, Hkv, d)); vv = np.zeros((n_slots, Hkv, d)); qq = np.zeros((n_slots, Hq, d))
    for ph, (pos, slot, req) in zip(wl.phases, run.positions):
        kk[slot] = ph.k_new; vv[slot] = ph.v_new
        if ph.q is not None:
            qq[slot] = ph.q
    last = wl.phases[-1].desc
    off = last["br_kv_off"]          # stage-1 branches 0..2, serial tokens between the stages, stage-2 branches 0..1
    flat_slot = ([0, 1, 2, 3, 4] + [off[0], off[1], off[2], off[0] + 1, off[2] + 1, off[0] + 2] + [off[3], off[3] + 1]
                 + [off[4], off[5], off[4] + 1] + [int(last["tail_off"][0])])
    assert len(flat_slot) == len(rows)
    branch = [r[1] for r in rows]; stage = [r[2] for r in rows]
    dense = oracle.dense_attn(qq[flat_slot], kk[flat_slot], vv[flat_slot], branch, stage, theta, wl.sm_scale)
    par, ser = run.outputs
    np.testing.assert_allclose(par[0], dense[15], atol=1e-12)       # second token of stage-2 branch 0
    np.testing.assert_allclose(par[1], dense[14], atol=1e-12)       # first token of stage-2 branch 1
    np.testing.assert_allclose(ser[0], dense[16], atol=1e-12)
    # positions and visible sets against the hand-derived table
    ph = [p for p in wl.phases if p.label == "parallel-step"][0]
    pos, slot, _ = oracle.new_tokens(ph.desc, oracle.MODE_BRANCH)
    assert pos.tolist() == [rows[15][3], rows[14][3]]
    vis = oracle.visible_slots(ph.desc, oracle.MODE_BRANCH, n_slots)
    for t, flat in enumerate((15, 14)):
        assert sorted(np.flatnonzero(vis[t]).tolist()) == sorted(int(flat_slot[j]) for j in rows[flat][4])
    pos, _, _ = oracle.new_tokens(wl.phases[-1].desc, oracle.MODE_SERIAL)
    assert pos.tolist() == [rows[16][3]]


def _variant_positions(wl, rule, k=32):
    """Position IDs of every phase under a position-ID variant of the paper's ablation (written
    here, in the test, from the variant's definition): "fix-k" gives branch b the pre-allocated
    interval starting at P + b*k; "same-max" keeps the shared IDs but lets the serial token resume
    right after the largest branch position."""
    out = []
    for ph in wl.phases:
        d = ph.desc
        P = int(d["prefix_len"][0])
        if ph.mode == W.MODE_BRANCH:
            pos = []
            for b in range(int(d["n_branches"][0])):
                kv, ql = int(d["br_kv_len"][b]), int(d["br_q_len"][b])
                start = P + (b * k if rule == "fix-k" and P > 0 else 0)
                pos += [start + kv - ql + i for i in range(max(ql, 0))]
            out.append(np.array(pos, dtype=np.int32))
        else:
            lens = [int(x) for x in d["br_kv_len"]]
            base = P + (max(lens) if rule == "same-max" else len(lens) * k)
            out.append(np.array([base + int(d["tail_len"][0]) - 1], dtype=np.int32))
    return out


def test_position_id_variants_through_caller_given_positions():
    """aspd_oracle_attn_at: with Eq. 4's own positions it is aspd_oracle_attn; with the ablation's
    variants each branch still equals a standalone causal sequence at the variant's positions
    (library SDPA), i.e. only the position IDs changed, not the mask."""
    wl = W.build_segment_workload("var", 17, 4, 2, 16, "f32", 1e4, [23], [[5, 2, 9]], [[1, 1, 1]], serial_steps=1)
    base = run_workload(wl)
    same = oracle.run.OracleRun(wl)
    for ph, (pos, _, _) in zip(wl.phases, base.positions):
        same.step(ph, pos_override=pos)
    for a, b in zip(base.outputs, same.outputs):
        np.testing.assert_array_equal(a, b)
    P, kpre, vpre, kb, vb, _ = _branch_tokens(wl)
    par = [p for p in wl.phases if p.label == "parallel-step"][0]
    for rule in ("fix-k", "same-max"):
        run = oracle.run.OracleRun(wl)
        for ph, pos in zip(wl.phases, _variant_positions(wl, rule)):
            run.step(ph, pos_override=pos)
        for b in range(3):
            start = P + (32 * b if rule == "fix-k" else 0)
            positions = np.concatenate([np.arange(P), start + np.arange(len(kb[b]))])
            ref = _sdpa_causal_last(par.q[b], np.concatenate([kpre, kb[b]]), np.concatenate([vpre, vb[b]]), positions,
                                    wl.theta, wl.sm_scale, wl.G)
            np.testing.assert_allclose(run.outputs[0][b], ref, atol=1e-10)
        assert not np.allclose(run.outputs[1], base.outputs[1])      # the serial token sits elsewhere


# ------------------------------------------------------------------ softmax closed forms
# ------------------------------------------------- the ablation's visible ("Shared") mask
GOLDEN_SHARED = os.path.join(os.path.dirname(__file__), "golden", "worked_example_shared_mask.txt")


def test_shared_mask_worked_example():
    """Hand-derived visible sets of the worked example when the visibility function is 1
    everywhere and only the order of the position IDs remains."""
    rows = load_example()
    pos = oracle.dense_positions([r[1] for r in rows], [r[2] for r in rows])
    vis = oracle.dense_visible_shared(pos)
    n = 0
    for line in open(GOLDEN_SHARED):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        idx, p_, want = line.split()
        assert int(p_) == pos[int(idx)]
        assert np.flatnonzero(vis[int(idx)]).tolist() == [int(x) for x in want.split(",")], idx
        n += 1
    assert n == len(rows)
    # a superset of the branch-invisible mask, equal to it on the main branch
    iso = oracle.dense_visible([r[1] for r in rows], [r[2] for r in rows])
    assert (vis >= iso).all() and (vis != iso).any()
    for i, r in enumerate(rows):
        if r[1] < 0:
            assert (vis[i] == iso[i]).all()


def test_shared_mask_is_what_exists_under_lockstep_decoding():
    """Another description of the same mask, by time instead of by position: a serial step decodes
    one token, a parallel step one token of every live branch; a token sees what earlier STEPS
    produced, and itself.  Random multi-stage requests; also the attention itself against library
    SDPA with that boolean mask."""
    rng = np.random.default_rng(19)
    for trial in range(30):
        branch, stage, born = [], [], []
        st, step = 0, 0
        for _seg in range(int(rng.integers(1, 4))):
            for _ in range(int(rng.integers(1, 5))):
                branch.append(-1); stage.append(st); born.append(step); step += 1
            st += 1
            lens = rng.integers(1, 5, size=int(rng.integers(1, 4)))
            for k in range(int(lens.max())):
                for b in range(len(lens)):
                    if k < lens[b]:
                        branch.append(b); stage.append(st); born.append(step)
                step += 1
            st += 1
        branch.append(-1); stage.append(st); born.append(step)
        L = len(branch)
        want = np.array([[1 if (born[j] < born[i] or i == j) else 0 for j in range(L)] for i in range(L)], dtype=np.uint8)
        pos = oracle.dense_positions(branch, stage)
        np.testing.assert_array_equal(oracle.dense_visible_shared(pos), want)
        if trial < 4:
            Hq, Hkv, d, theta, scale = 4, 2, 8, 77.0, 0.3
            q = rng.standard_normal((L, Hq, d)); k = rng.standard_normal((L, Hkv, d)); v = rng.standard_normal((L, Hkv, d))
            out = oracle.dense_attn(q, k, v, branch, stage, theta, scale, mask=oracle.MASK_SHARED)
            qh = torch.tensor(_library_rotary(q, pos, theta)).permute(1, 0, 2)
            kh = torch.tensor(_library_rotary(k, pos, theta)).permute(1, 0, 2).repeat_interleave(Hq // Hkv, dim=0)
            vv = torch.tensor(v).permute(1, 0, 2).repeat_interleave(Hq // Hkv, dim=0)
            ref = torch.nn.functional.scaled_dot_product_attention(qh[None], kh[None], vv[None],
                                                                   attn_mask=torch.tensor(want.astype(bool)), scale=scale)
            np.testing.assert_allclose(out, ref[0].permute(1, 0, 2).numpy(), atol=1e-12)


def test_shared_mask_descriptor_visible_sets():
    """Descriptor form, integers: a new token at offset k of its branch sees the prefix, earlier
    stages, its own branch up to itself and the first k tokens of every other branch of its
    stage -- also of branches that decode nothing in this step."""
    wl = W.build_two_stage_workload("ts", 5, 4, 2, 8, "f32", 1e4, 7, [3, 1, 2], 2, [4, 0, 6], [1, 2, 1])
    ph = [p for p in wl.phases if p.mode == W.MODE_BRANCH and p.q is not None][-1]
    d = ph.desc
    n_slots = int(d["n_pages"][0]) * wl.page_size
    vis = oracle.visible_slots(d, oracle.MODE_BRANCH, n_slots, mask=oracle.MASK_SHARED)
    iso = oracle.visible_slots(d, oracle.MODE_BRANCH, n_slots)
    t = 0
    for b in range(int(d["n_branches"][0])):
        for i in range(max(0, int(d["br_q_len"][b]))):
            k = int(d["br_kv_len"][b]) - int(d["br_q_len"][b]) + i
            extra = set()
            for c in range(int(d["n_branches"][0])):
                if c != b and int(d["br_q_len"][c]) >= 0:
                    extra |= {int(d["br_kv_off"][c]) + j for j in range(min(k, int(d["br_kv_len"][c])))}
            assert set(np.flatnonzero(vis[t])) == set(np.flatnonzero(iso[t])) | extra, (b, i)
            t += 1
    assert t == len(vis) and (vis != iso).any()


def _load_shared_example():
    rows = {}
    for line in open(GOLDEN_SHARED):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        idx, p_, want = line.split()
        rows[int(idx)] = (int(p_), [int(x) for x in want.split(",")])
    return rows


def test_shared_mask_descriptor_matches_worked_example():
    """The descriptor form under the visible mask against the hand-derived table, mapped to slots the
    way the paper's mask is: rows 8 and 9 (second step of stage 1: two live branches at offset 1, one
    stopped branch of one token), row 10 (last step of stage 1: offset 2, the others stopped), row 15
    (stage 3: offset 1, the other branch stopped at one token) and row 16 (the serial token after it,
    the same under both masks)."""
    rows = _load_shared_example()
    # ---- stage 1, its second decoding step: branches 0 and 2 decode their second token
    wl = W.build_segment_workload("t", 1, 2, 1, 8, "f32", 100.0, [5], [[1, 1, 1]], [[1, 0, 1]])
    par = [p for p in wl.phases if p.label == "parallel-step"][0]
    pos, _, _ = oracle.new_tokens(par.desc, oracle.MODE_BRANCH)
    assert pos.tolist() == [rows[8][0], rows[9][0]]
    n_slots = int(par.desc["n_pages"][0]) * wl.page_size
    off = par.desc["br_kv_off"]
    flat_to_slot = {i: i for i in range(5)}
    flat_to_slot.update({5: off[0], 8: off[0] + 1, 10: off[0] + 2, 6: off[1], 7: off[2], 9: off[2] + 1})
    vis = oracle.visible_slots(par.desc, oracle.MODE_BRANCH, n_slots, mask=oracle.MASK_SHARED)
    for t, flat in enumerate((8, 9)):
        assert sorted(np.flatnonzero(vis[t]).tolist()) == sorted(int(flat_to_slot[j]) for j in rows[flat][1]), flat
    # ---- stage 1, its last step: only branch 0 decodes (offset 2); it sees both tokens of branch 2
    wl = W.build_segment_workload("t", 1, 2, 1, 8, "f32", 100.0, [5], [[2, 1, 2]], [[1, 0, 0]])
    par = [p for p in wl.phases if p.label == "parallel-step"][0]
    pos, _, _ = oracle.new_tokens(par.desc, oracle.MODE_BRANCH)
    assert pos.tolist() == [rows[10][0]]
    assert (par.desc["br_kv_off"] == off).all()
    vis = oracle.visible_slots(par.desc, oracle.MODE_BRANCH, n_slots, mask=oracle.MASK_SHARED)
    assert sorted(np.flatnonzero(vis[0]).tolist()) == sorted(int(flat_to_slot[j]) for j in rows[10][1])
    # ---- stage 3 (a second parallel stage) and the serial token after it
    wl = W.build_two_stage_workload("t2", 3, 2, 1, 8, "f32", 100.0, 5, [3, 1, 2], 2, [1, 1], [1, 0], serial_steps=1)
    par = [p for p in wl.phases if p.label == "parallel-step"][0]
    d = par.desc
    pos, _, _ = oracle.new_tokens(d, oracle.MODE_BRANCH)
    assert pos.tolist() == [rows[15][0]]
    off = d["br_kv_off"]      # regions: stage-1 branches 0..2, the two serial tokens, stage-3 branches 0..1
    flat_to_slot = {i: i for i in range(5)}
    flat_to_slot.update({5: off[0], 8: off[0] + 1, 10: off[0] + 2, 6: off[1], 7: off[2], 9: off[2] + 1,
                         11: off[3], 12: off[3] + 1, 13: off[4], 15: off[4] + 1, 14: off[5]})
    n_slots = int(d["n_pages"][0]) * wl.page_size
    vis = oracle.visible_slots(d, oracle.MODE_BRANCH, n_slots, mask=oracle.MASK_SHARED)
    assert sorted(np.flatnonzero(vis[0]).tolist()) == sorted(int(flat_to_slot[j]) for j in rows[15][1])
    iso = oracle.visible_slots(d, oracle.MODE_BRANCH, n_slots)
    assert set(np.flatnonzero(vis[0])) - set(np.flatnonzero(iso[0])) == {int(off[5])}      # flat index 14 is what the mask adds
    ser = [p for p in wl.phases if p.label == "serial-0"][0]
    pos, _, _ = oracle.new_tokens(ser.desc, oracle.MODE_SERIAL)
    assert pos.tolist() == [rows[16][0]]
    flat_to_slot[16] = int(ser.desc["tail_off"][0])
    vis = oracle.visible_slots(ser.desc, oracle.MODE_SERIAL, n_slots, mask=oracle.MASK_SHARED)
    assert sorted(np.flatnonzero(vis[0]).tolist()) == sorted(int(flat_to_slot[j]) for j in rows[16][1])


def test_shared_mask_single_branch_is_plain_causal():
    """With one branch there is nobody else to see: both masks give the same attention."""
    wl = W.build_segment_workload("one", 9, 4, 2, 16, "f32", 1e4, [11], [[5]], [[3]], serial_steps=1)
    a, b = run_workload(wl), run_workload(wl, oracle.MASK_SHARED)
    for x, y in zip(a.outputs, b.outputs):
        np.testing.assert_array_equal(x, y)


def test_softmax_closed_forms():
    wl = W.build_segment_workload("c", 21, 4, 2, 16, "f32", 10000.0, [19], [[4, 9]], [[1, 1]], serial_steps=1)
    ph = {p.label: p for p in wl.phases}
    # (i) constant V => output is that constant
    run = oracle.run.OracleRun(wl)
    for p in wl.phases:
        p.v_new[:] = 0.75
    for p in wl.phases:
        o = run.step(p)
        if o is not None:
            np.testing.assert_allclose(o, 0.75, atol=1e-13)
    # (ii) all keys zero => uniform weights => mean of the visible V (sets from the prose:
    #      prefix + own branch; serial: everything)
    wl = W.build_segment_workload("c", 21, 4, 2, 16, "f32", 10000.0, [19], [[4, 9]], [[1, 1]], serial_steps=1)
    ph = {p.label: p for p in wl.phases}
    for p in wl.phases:
        p.k_new[:] = 0.0
    run = run_workload(wl)
    vpre = ph["fill-prefix"].v_new.astype(np.float64)
    vb = ph["fill-branches"].v_new.astype(np.float64)
    vn = ph["parallel-step"].v_new.astype(np.float64)
    sets = [np.concatenate([vpre, vb[:4], vn[0:1]]), np.concatenate([vpre, vb[4:13], vn[1:2]])]
    for b in range(2):
        for h in range(4):
            np.testing.assert_allclose(run.outputs[0][b, h], sets[b][:, h // 2, :].mean(axis=0), atol=1e-12)
    everything = np.concatenate([vpre, vb, vn, ph["serial-0"].v_new.astype(np.float64)])
    assert len(everything) == 19 + 5 + 10 + 1
    for h in range(4):
        np.testing.assert_allclose(run.outputs[1][0, h], everything[:, h // 2, :].mean(axis=0), atol=1e-12)
    # (iii) one key with a huge logit => output is (almost) its V
    wl = W.build_segment_workload("c", 22, 2, 2, 16, "f32", 10000.0, [19], [[4]], [[1]])
    ph = {p.label: p for p in wl.phases}
    qn = ph["parallel-step"].q
    target = 7                                   # prefix token at position 7, query at position 23
    for h in range(2):
        # k = un-rotate(rotate(q, 23), 7) * big  =>  q_hat . k_hat = big * |q|^2 (logits far beyond
        # exp's range unless the maximum is subtracted first)
        qh = oracle.rope(qn[0, h], 23.0, wl.theta)
        # inverse rotation = rotation by the negative position
        ph["fill-prefix"].k_new[target, h] = (oracle.rope(qh, -7.0, wl.theta) * 400.0).astype(np.float32)
    run = run_workload(wl)
    np.testing.assert_allclose(run.outputs[0][0], ph["fill-prefix"].v_new[target], atol=1e-6)


# ------------------------------------------------------------------------- paged append
def test_paged_append_lands_where_the_page_table_says():
    wl = W.build_segment_workload("pg", 31, 2, 2, 8, "f32", 10000.0, [15, 17], [[16, 1], [17]], [[1, 1], [1]],
                                  serial_steps=1)
    run = run_workload(wl)
    seen = set()
    for ph, (pos, slot, req) in zip(wl.phases, run.positions):
        for t in range(len(pos)):
            r = int(req[t]); s = int(slot[t])
            page = int(ph.desc["page_ids"][int(ph.desc["page_begin"][r]) + s // wl.page_size])
            row = s % wl.page_size
            assert (page, row) not in seen
            seen.add((page, row))
            np.testing.assert_array_equal(run.v_pool[page, :, row, :], ph.v_new[t])
            for h in range(wl.Hkv):
                np.testing.assert_allclose(run.k_pool[page, h, row], oracle.rope(ph.k_new[t, h], float(pos[t]), wl.theta),
                                           atol=0)
    # untouched rows stay zero
    total = sum(len(p[0]) for p in run.positions)
    assert int((np.abs(run.v_pool).sum(axis=(1, 3)) > 0).sum()) == total
