"""Shared helpers of the GPU parity tests: upload of generated inputs and the
comparison rules between the CUDA path and the oracle."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2408_15562_b200 import binding, synth

NEAR = 1e-6          # relative width of the decision-boundary band that is counted, not failed


def make_ctx(inp: synth.VerifyInputs, n_layers=None, max_batch=None, max_nodes=None) -> binding.Context:
    w = inp.workload
    return binding.Context(w.n_q_heads, w.n_kv_heads, w.vocab, inp.max_len,
                           max_nodes=max_nodes or inp.parent.shape[1],
                           n_layers=n_layers or w.n_layers, max_batch=max_batch or w.batch)


def dev(a, dtype=None):
    if a is None:
        return None
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.to(dtype)
    return t.cuda()


def upload_attn(inp: synth.VerifyInputs):
    b = binding.bf16_tensor
    return dict(q=b(inp.q), k_cache=b(inp.k_cache), v_cache=b(inp.v_cache), tree_k=b(inp.tree_k),
                tree_v=b(inp.tree_v), parent=dev(inp.parent), prefix_len=dev(inp.prefix_len))


def upload_accept(inp: synth.VerifyInputs):
    return dict(target_logits=dev(inp.target_logits), draft_probs=dev(inp.draft_probs),
                draft_tokens=dev(inp.draft_tokens), parent=dev(inp.parent),
                temperature=dev(inp.temperature),
                uniforms=dev(inp.uniforms) if inp.draft_probs is not None else None)


def attn_errors(gpu_out: torch.Tensor, ref: np.ndarray):
    got = gpu_out.float().cpu().numpy().astype(np.float64)
    err = np.abs(got - ref)
    return float(err.max()), float(err.mean())


def compare_accept(inp: synth.VerifyInputs, path, n_acc, bonus, seqs=None):
    """Compare the CUDA acceptance result with the oracle, sequence by sequence.

    Returns (hard_mismatches, near_boundary_count, messages).  A divergence is
    tolerated only if the oracle's fp64 values put the decision within NEAR of
    its boundary; the oracle is then re-run forced onto the CUDA branch and the
    rest of the walk must agree.
    """
    path = np.asarray(path)
    n_acc = np.asarray(n_acc)
    bonus = np.asarray(bonus)
    B, N = inp.parent.shape
    hard, near, msgs = 0, 0, []
    for b in (range(B) if seqs is None else seqs):
        sl = slice(b, b + 1)
        dp = None if inp.draft_probs is None else inp.draft_probs[sl]
        un = inp.uniforms[sl] if dp is not None else None
        force = np.full((1, N), -1, np.int32)
        g_path = [int(x) for x in path[b, :int(n_acc[b])]]
        ok = False
        for _ in range(N + 2):
            r = oracle.tree_accept(inp.target_logits[sl], dp, inp.draft_tokens[sl], inp.parent[sl],
                                   inp.temperature[sl], un, force)
            o_path = [int(x) for x in r["accepted_path"][0, :int(r["n_accepted"][0])]]
            if o_path == g_path:
                if int(r["bonus_token"][0]) == int(bonus[b]):
                    ok = True
                else:
                    info = r["bonus_info"][0]
                    uz, lo, hi, Z, prv, nxt = info
                    g = int(bonus[b])
                    near_lo = abs(uz - lo) <= NEAR * Z and g == int(prv)
                    near_hi = abs(uz - hi) <= NEAR * Z and g == int(nxt)
                    if inp.temperature[b] > 0 and (near_lo or near_hi):
                        near += 1
                        ok = True
                        msgs.append("seq %d: bonus within band (oracle %d, cuda %d)" % (b, int(r["bonus_token"][0]), g))
                    else:
                        msgs.append("seq %d: bonus mismatch oracle %d cuda %d info %s" % (b, int(r["bonus_token"][0]), g, info))
                break
            # first child on which the two walks decided differently
            tested = [c for c in range(1, N) if not np.isnan(r["trace_rq"][0, c])] if inp.temperature[b] > 0 else []
            diff = None
            for c in tested:
                if (c in o_path) != (c in g_path):
                    diff = c
                    break
            if diff is None:
                msgs.append("seq %d: path mismatch oracle %s cuda %s" % (b, o_path, g_path))
                break
            rq, p = r["trace_rq"][0, diff], r["trace_p"][0, diff]
            if abs(rq - p) <= NEAR * max(rq, p):
                near += 1
                force[0, diff] = 1 if diff in g_path else 0
                msgs.append("seq %d: node %d within band (rq=%r p=%r)" % (b, diff, rq, p))
                continue
            msgs.append("seq %d: decision mismatch at node %d rq=%r p=%r oracle %s cuda %s" % (b, diff, rq, p, o_path, g_path))
            break
        if not ok:
            hard += 1
        if (path[b, int(n_acc[b]):] != -1).any():
            hard += 1
            msgs.append("seq %d: path padding is not -1" % b)
    return hard, near, msgs
