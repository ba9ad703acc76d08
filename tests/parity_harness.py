"""Lock-step comparison of the CUDA library (through its C ABI) with the fp64 oracle.

Used by the GPU parity tests and by the smoke check.  Acceptance rules:
  * attention output: max |gpu - ref| over a head's row <= tol * max |ref| of that row
    (tol 1e-5 for fp32 caches, 2e-3 for bf16 caches; a bf16 `out` additionally gets
    half a bf16 ulp of the row maximum, 2^-9, the rounding of the store itself);
  * importance scores: |gpu - ref| <= 1e-4 * ref + 2^-100 on every live token.  The absolute
    term is the flush rule: the GPU forms probabilities in fp32 and one below 2^-126 becomes
    zero, while the fp64 oracle keeps it; a score can therefore be short by (steps) * 2^-126,
    and scores that small are equal for every purpose of the method;
  * teacher-forced selection: the oracle's select() fed the GPU's own fp32 scores and
    position ids returns exactly the GPU's evicted position ids (integer work: bit exact);
  * free-running: where the oracle's own choice differs from the GPU's, every token in
    the symmetric difference must have an oracle score within 1e-5 relative of the
    cutoff (plus the same 2^-100: tokens whose scores were flushed to zero on the GPU tie
    there and go by position id); such events are counted and the oracle is then forced to
    the GPU's choice so the comparison stays in lock-step.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

import paper_2605_29873_b200 as mkv
from oracle import mkv_oracle as O
from workloads.synthetic import BatchStream, Workload


FLUSH_ATOL = 2.0 ** -100   # see the module doc: fp32 probabilities below 2^-126 are flushed to zero


@dataclass
class ParityReport:
    steps: int = 0
    max_out_err: float = 0.0
    max_score_err: float = 0.0
    evictions: int = 0
    evicted_not_newest: int = 0
    near_ties: int = 0
    failures: list = field(default_factory=list)

    def ok(self):
        return not self.failures


def to_device(arr, torch, dtype, device):
    """fp64 numpy values that already lie on the dtype's grid -> device tensor (exact)."""
    return torch.from_numpy(np.ascontiguousarray(arr, dtype=np.float32)).to(device=device, dtype=dtype)


def make_context(w: Workload, kernel=mkv.MKV_KERNEL_AUTO, out_f32=True, sequences=None, record_probs=False,
                 budget_max=None, layers=1, score_mode=mkv.MKV_SCORE_GROUP_MEAN, flags=0):
    batch = w.batch if sequences is None else len(sequences)
    kv_dtype = mkv.MKV_BF16 if w.dtype == "bf16" else mkv.MKV_F32
    out_dtype = mkv.MKV_F32 if (out_f32 or kv_dtype == mkv.MKV_F32) else mkv.MKV_BF16
    lens = w.prefill_lens() if sequences is None else w.prefill_lens()[list(sequences)]
    return mkv.MomentKV(layers, w.q_heads, w.kv_heads, w.head_dim, budget_max or w.budget, w.beta, batch,
                        int(max(lens.max(), 1)), kv_dtype=kv_dtype, out_dtype=out_dtype, kernel=kernel, score_mode=score_mode,
                        flags=flags | (mkv.MKV_FLAG_RECORD_PROBS if record_probs else 0))


def prefill_both(ctx, w: Workload, stream: BatchStream, layer=0, mode=O.GROUP_MEAN, budget=None):
    torch = ctx.torch
    Ks, Vs = stream.prefill()
    lens = stream.lens
    B, src = len(Ks), int(max(lens.max(), 1))
    Kpad = np.zeros((B, w.kv_heads, src, w.head_dim))
    Vpad = np.zeros_like(Kpad)
    for b in range(B):
        Kpad[b, :, : lens[b]] = Ks[b]
        Vpad[b, :, : lens[b]] = Vs[b]
    dt = ctx.torch_kv_dtype()
    ctx.prefill(layer, to_device(Kpad, torch, dt, ctx.device), to_device(Vpad, torch, dt, ctx.device), lens)
    oracles = [O.OracleSequence(w.q_heads, w.kv_heads, w.head_dim, budget or w.budget, w.beta, int(lens[b]), mode)
               for b in range(B)]
    for b in range(B):
        oracles[b].prefill(Ks[b], Vs[b])
    return oracles, (Ks, Vs)


def lockstep(ctx, w: Workload, stream: BatchStream, oracles, steps, layer=0, report: ParityReport | None = None,
             check_state_every=1, chunk=64, host_api=False, host_packed=False, host_pinned=True, tol_out=None,
             tol_score=1e-4):
    """Runs `steps` decode steps on both sides, comparing as described in the module doc.
    tol_out / tol_score replace the standard tolerances (only the test of extreme logits does)."""
    torch = ctx.torch
    rep = report or ParityReport()
    B = len(oracles)
    dt, odt = ctx.torch_kv_dtype(), ctx.torch_out_dtype()
    if tol_out is None:
        tol_out = 1e-5 if w.dtype == "f32" else 2e-3
    out = torch.zeros((B, w.q_heads, w.head_dim), dtype=odt, device=ctx.device)
    done = 0
    while done < steps:
        nb = min(chunk, steps - done)
        qs, ks, vs = stream.next(nb)
        if host_api:
            pin = (lambda t: t.pin_memory()) if host_pinned else (lambda t: t)   # pageable: the staged path
            qd = pin(to_device(qs, torch, dt, "cpu"))
            kd = pin(to_device(ks, torch, dt, "cpu"))
            vd = pin(to_device(vs, torch, dt, "cpu"))
            if host_packed:      # q | k_new | v_new of a step back to back: the single-copy path
                nq, nk = qd[0].numel(), kd[0].numel()
                pk = pin(torch.empty((nb, nq + 2 * nk), dtype=dt))
                pk[:, :nq] = qd.reshape(nb, -1); pk[:, nq:nq + nk] = kd.reshape(nb, -1); pk[:, nq + nk:] = vd.reshape(nb, -1)
                qd = [pk[j, :nq] for j in range(nb)]
                kd = [pk[j, nq:nq + nk] for j in range(nb)]
                vd = [pk[j, nq + nk:] for j in range(nb)]
            out_h = pin(torch.zeros((B, w.q_heads, w.head_dim), dtype=odt))
        else:
            qd, kd, vd = (to_device(a, torch, dt, ctx.device) for a in (qs, ks, vs))
        for i in range(nb):
            t = oracles[0].steps_done()
            if host_api:
                ctx.decode_step_host(layer, qd[i], kd[i], vd[i], out_h)
                torch.cuda.synchronize()
                got = out_h.to(torch.float64).numpy()
            else:
                ctx.decode_step(layer, qd[i], kd[i], vd[i], out)
                got = out.to(torch.float64).cpu().numpy()
            check_state = (check_state_every > 0 and (rep.steps % check_state_every == 0))
            for b in range(B):
                ref = oracles[b].attend_update(qs[i, b], ks[i, b], vs[i, b])
                rowmax = np.abs(ref).max(axis=1)
                err = np.abs(got[b] - ref).max(axis=1)
                allow = tol_out * rowmax
                if odt == torch.bfloat16:
                    allow = allow + rowmax * 2.0 ** -9
                rel = float((err / np.maximum(rowmax, 1e-300)).max())
                rep.max_out_err = max(rep.max_out_err, rel)
                if (err > allow).any():
                    rep.failures.append(f"step {t} seq {b}: out error {rel:.3e}")
                for g in range(w.kv_heads):
                    o_choice = oracles[b].choose(g)
                    if not check_state and len(o_choice) == 0:
                        continue
                    ev_pos, ev_sc = ctx.last_evicted(layer, b, g)
                    forced = None
                    if check_state or len(ev_pos) != len(o_choice) or set(ev_pos.tolist()) != set(o_choice.tolist()):
                        g_pos, g_sc = ctx.decode_state(layer, b, g)
                        all_pos = np.concatenate([g_pos, ev_pos]).astype(np.int64)
                        all_sc = np.concatenate([g_sc, ev_sc]).astype(np.float64)
                        o_pos, o_sc, _ = oracles[b].decode_state(g)
                        if sorted(all_pos.tolist()) != sorted(o_pos.tolist()):
                            rep.failures.append(f"step {t} unit ({b},{g}): token sets differ")
                            continue
                        order = np.argsort(all_pos)
                        oorder = np.argsort(o_pos)
                        sdiff = np.abs(all_sc[order] - o_sc[oorder])
                        serr = np.maximum(sdiff - FLUSH_ATOL, 0.0) / np.maximum(o_sc[oorder], 1e-300)
                        rep.max_score_err = max(rep.max_score_err, float(serr.max()))
                        if serr.max() > tol_score:
                            rep.failures.append(f"step {t} unit ({b},{g}): score error {serr.max():.3e}")
                        # teacher-forced: integer selection on the GPU's own scores
                        k = len(ev_pos)
                        want = all_pos[O.select(all_sc, all_pos, k)] if k else np.zeros(0, dtype=np.int64)
                        if sorted(want.tolist()) != sorted(ev_pos.tolist()):
                            rep.failures.append(f"step {t} unit ({b},{g}): selection differs from select() on GPU scores")
                        if k != len(o_choice):
                            rep.failures.append(f"step {t} unit ({b},{g}): evicted {k}, oracle {len(o_choice)}")
                        elif set(ev_pos.tolist()) != set(o_choice.tolist()):
                            # free-running difference: tolerated only as a near tie at the cutoff
                            cutoff = np.sort(o_sc)[k - 1]
                            diff = set(ev_pos.tolist()) ^ set(o_choice.tolist())
                            smap = dict(zip(o_pos.tolist(), o_sc.tolist()))
                            worst = max(max(abs(smap[p] - cutoff) - FLUSH_ATOL, 0.0) / max(cutoff, 1e-300) for p in diff)
                            if worst <= 1e-5:
                                rep.near_ties += 1
                            else:
                                rep.failures.append(f"step {t} unit ({b},{g}): eviction differs, gap {worst:.3e}")
                            forced = ev_pos
                    if len(ev_pos):
                        rep.evictions += 1
                        rep.evicted_not_newest += int(t not in ev_pos.tolist())
                    if forced is not None:
                        oracles[b]._forced = getattr(oracles[b], "_forced", {})
                        oracles[b]._forced[g] = forced
                fz = getattr(oracles[b], "_forced", None)
                if fz:
                    force = [fz.get(g, oracles[b].choose(g)).astype(np.int64) for g in range(w.kv_heads)]
                    oracles[b].evict(force=force)
                    oracles[b]._forced = {}
                else:
                    oracles[b].evict()
            rep.steps += 1
            if len(rep.failures) > 20:
                return rep
        done += nb
    ctx.status_sync()
    return rep
