"""Shared driver of the parity tests: runs one DES step on the CPU oracle and
on the CUDA library (through the C ABI binding) from the same seeded batch, and
compares everything the step produces.

Tolerances
  integer outputs (shards, rows, unique indices, key set, init bits): exact;
  float32 forward outputs: |d| <= 1e-5 |ref| + 1e-6 + 2e-6 * sum_j |t_j| for the
    per-sample sums (M_1 of LR and FM, A, R_lr): in the multi-hot workloads one
    hot id occurs hundreds of times in a sample, its row is added again and
    again to a growing float32 accumulator, and when the other terms cancel the
    (small) result cannot stay within 1e-5 of itself in float32; the last term
    measures the error against the size of the summands instead (condition-
    aware bound; it is zero-cost for the well-conditioned elements);
  summed per-key gradients G: |dG| <= 1e-5 |G| + 1e-6 + 2e-7 * sum_j |g_j|: a hot
    key sums thousands of O(1) terms of both signs; the scatter keeps every
    float32 chain to a few hundred additions and combines them in double, hence
    the ten times smaller constant.
  updated weights / optimizer state: the forward tolerance plus what dG does to
    ONE optimizer application (SGD: lr dG; Adagrad: lr dG / (sqrt(acc) + eps)
    for the weight, 2|G| dG + dG^2 for the accumulator) — Adagrad divides by
    sqrt(acc), so a gradient that cancels to ~eps moves the weight by O(lr)
    for a rounding-sized dG;
  anything downstream of the bf16 first-layer GEMM: 2e-2 relative plus 1e-3 of
    the tensor's largest magnitude (elements that cancel to ~0).
After every step the CUDA table's touched rows are overwritten with the
oracle's (des_table_write_rows), so each step is compared from identical state
and tolerated differences do not compound; `resync=False` keeps the drift."""
from __future__ import annotations

import numpy as np
import torch

from oracle import Oracle
from paper_1909_04823_b200 import synth
from paper_1909_04823_b200.synth import OP_DENSE1, OP_FM, OP_LR, OP_POOL, PART_FIELD

RTOL, ATOL, SUMTOL, SUMTOL_FWD = 1e-5, 1e-6, 2e-7, 2e-6


# Per output: how many compared elements were outside the STATED bound rtol |ref| + atol (before the
# condition-aware term), out of how many, the worst condition number sum|t| / |sum t| among those, and their
# worst error in units of the stated bound.  Filled by close32 whenever it is given the extra term; the
# full-size tests assert caps on it and conftest writes it out when DES_TOL_REPORT names a file.
TOL_STATS = {}
TOL_CONTEXT = [""]          # label of the workload being compared (set by Pair.step)


def close32(got, ref, what, rtol=RTOL, atol=ATOL, extra=None, sumabs=None):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape, (what, got.shape, ref.shape)
    err = np.abs(got - ref)
    tol = rtol * np.abs(ref) + atol
    if extra is not None:
        out = err > tol
        st = TOL_STATS.setdefault(f"{TOL_CONTEXT[0]}: {what}", dict(outside_stated=0, total=0, worst_cond=0.0, worst_over=0.0))
        st["outside_stated"] += int(out.sum()); st["total"] += int(err.size)
        if out.any():
            st["worst_over"] = max(st["worst_over"], float((err[out] / tol[out]).max()))
            if sumabs is not None:
                sa = np.broadcast_to(np.asarray(sumabs, dtype=np.float64), err.shape)
                st["worst_cond"] = max(st["worst_cond"], float((sa[out] / np.maximum(np.abs(ref[out]), 1e-300)).max()))
        tol = tol + extra
    if not np.all(err <= tol):
        i = np.unravel_index(np.argmax(err - tol), err.shape)
        raise AssertionError(f"{what}: worst at {i}: got {got[i]!r} ref {ref[i]!r} err {err[i]:.3e} tol {tol[i]:.3e}; "
                             f"{int((err > tol).sum())} of {err.size} out of tolerance")


def close_gemm(got, ref, what, extra=None, sumabs=None):
    ref = np.asarray(ref, dtype=np.float64)
    close32(got, ref, "[gemm] " + what, rtol=2e-2, atol=1e-3 * max(float(np.abs(ref).max()), 1e-30), extra=extra,
            sumabs=sumabs)


def u32(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().numpy().view(np.uint32)


def select_samples(batch, idx):
    """A batch made of the given samples of `batch`, in the given order."""
    F = batch.fields
    lo = batch.offsets[np.asarray(idx) * F]
    hi = batch.offsets[np.asarray(idx) * F + F]
    pos = np.concatenate([np.arange(a, b_) for a, b_ in zip(lo, hi)]) if len(idx) else np.zeros(0, np.int64)
    lens = np.concatenate([np.diff(batch.offsets[i * F:i * F + F + 1]) for i in idx])
    off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    return synth.Batch(len(idx), F, off, batch.ids[pos], None if batch.vals is None else batch.vals[pos])


def rows_per_shard_for(w, cap_total):
    """Row capacity per shard: even under HASH; by field vocabulary under FIELD."""
    if w.partition != PART_FIELD:
        return None
    per_field = []
    for f in range(w.fields):
        per_field.append(64 if f < w.bucket_fields else cap_total // max(1, w.fields - w.bucket_fields))
    out = [256] * w.shards
    for f, n in enumerate(per_field):
        out[f % w.shards] += int(n * 1.05) + 64
    return out


class Pair:
    """Oracle table + CUDA table for one workload."""

    def __init__(self, w, max_rows, max_nnz, max_batch=None, max_uniq=0, resync=True, omp=False):
        """omp: use the all-cores build of the oracle (the same source compiled with -fopenmp, pinned equal to the
        sequential build by tests/test_oracle_pins.py) — only for runs the sequential build would take minutes for."""
        from paper_1909_04823_b200.binding import Table
        self.w = w
        self.o = Oracle.for_workload(w, omp=omp)
        self.t = Table.for_workload(w, max_rows=max_rows, max_nnz=max_nnz, max_batch=max_batch or w.batch,
                                    rows_per_shard=rows_per_shard_for(w, max_rows), max_uniq=max_uniq)
        self.row_base = np.array(self.t.row_base(), dtype=np.int64)
        self.resync = resync
        self.drifted = False        # True once un-resynced differences may have accumulated
        self.nstep = 0              # backward calls so far (Adam's bias-correction step)
        if w.hidden:
            W1 = synth.dense1_weights(w)
            self.o.dense1_set(W1)
            self.t.dense1_set(torch.from_numpy(W1).cuda())

    def close(self):
        self.t.close(); self.o.close()

    # ------------------------------------------------------------------
    def insert_only(self, batch):
        from paper_1909_04823_b200.binding import DeviceBatch
        fi = self.o.find_or_insert(batch)
        db = DeviceBatch.from_synth(batch)
        self.t.find_or_insert(db, True)
        self.compare_index(batch, fi, db)
        return fi, db

    def compare_index(self, batch, fi, db, by_key=False):
        """by_key: the oracle's table holds only the keys of this batch (the CUDA table
        is pre-populated with many more), so row NUMBERS differ by construction; shards
        and batch-unique indices must still be identical, and rows are then compared
        through the unique index, i.e. key by key."""
        n = batch.nnz
        assert self.t.status() == 0
        assert np.array_equal(db.shards.cpu().numpy()[:n], fi["shards"]), "shards"
        assert np.array_equal(u32(db.uidx)[:n], fi["uidx"]), "uidx"
        U = int(db.n_uniq.item())
        assert U == fi["U"], ("n_uniq", U, fi["U"])
        if by_key:
            return
        assert np.array_equal(u32(db.rows)[:n], fi["rows"]), "rows"
        want = self.row_base[fi["uniq_shard"].astype(np.int64)] + fi["uniq_row"].astype(np.int64)
        assert np.array_equal(u32(db.uniq_rows)[:U].astype(np.int64), want), "uniq_rows"
        assert self.t.size() == [int(v) for v in self.o.size()], "table size"

    def _adam_tol(self, G, dG, m, v):
        """Bounds on |d theta|, |d m|, |d v| of one Adam application when the summed gradient moves
        by at most dG; m, v: the oracle's moments AFTER the application."""
        w, t = self.w, max(self.nstep, 1)
        c1, c2 = 1.0 - w.beta1 ** t, 1.0 - w.beta2 ** t
        dm = (1.0 - w.beta1) * dG
        dv = (1.0 - w.beta2) * (2.0 * np.abs(G) * dG + dG * dG)
        rt = np.sqrt(v / c2)
        drt = np.minimum(dv / c2 / (2.0 * rt + 1e-300), np.sqrt(dv / c2))
        den = rt + w.eps
        r = np.abs(m) / c1 / den
        dth = 2.0 * (dm / c1 / den + r * drt / den)
        return w.lr * np.minimum(dth, 2.0 * r + 2.0), dm, dv

    def _ftrl_tol(self, G, dG, w_old, w_new, n_new):
        """Bounds on |d w|, |d n|, |d z| of one FTRL-Proximal application."""
        w = self.w
        dn = 2.0 * np.abs(G) * dG + dG * dG
        rt = np.sqrt(n_new)
        drt = np.minimum(dn / (2.0 * rt + 1e-300), np.sqrt(dn))
        dz = dG + drt / w.ftrl_alpha * np.abs(w_old)
        D = (w.ftrl_beta + rt) / w.ftrl_alpha + w.ftrl_l2
        dw = 2.0 * (dz / D + np.abs(w_new) * (drt / w.ftrl_alpha) / D)
        return dw, dn, dz

    def compare_rows(self, fi, db, exact=False, gemm=False, what="rows", G=None, before=None):
        U = fi["U"]
        w = self.w
        ref = self.o.read_rows(fi["uniq_shard"], fi["uniq_row"])
        got = self.t.read_rows(db.uniq_rows[:U])
        adam = w.optimizer == synth.OPT_ADAM
        ftrl = w.lin_optimizer == synth.LIN_FTRL
        if adam or ftrl:
            ref.update(self.o.read_state2(fi["uniq_shard"], fi["uniq_row"]))
            got.update(self.t.read_state2(db.uniq_rows[:U]))
        torch.cuda.synchronize()
        sgd = w.optimizer == synth.OPT_SGD
        names = ["emb", "lin", "acc_emb", "acc_lin"] + (["acc2_emb"] if adam else []) + (["lin2"] if adam or ftrl else [])
        tol = {}
        if G is not None:
            for emb in (True, False):
                Gk = (G["Gv"] if emb else G["Gw"]).astype(np.float64)
                dG = RTOL * np.abs(Gk) + ATOL + SUMTOL * (G["Sv"] if emb else G["Sw"])
                if gemm:
                    dG = dG + 2e-2 * np.abs(Gk) + 1e-3 * max(float(np.abs(Gk).max()), 1e-30)
                th, s1, s2 = ("emb", "acc_emb", "acc2_emb") if emb else ("lin", "acc_lin", "lin2")
                if ftrl and not emb:
                    tol[th], tol[s1], tol[s2] = self._ftrl_tol(Gk, dG, before["lin"].astype(np.float64),
                                                               ref["lin"].astype(np.float64),
                                                               ref["acc_lin"].astype(np.float64))
                elif adam:
                    tol[th], tol[s1], tol[s2] = self._adam_tol(Gk, dG, ref[s1].astype(np.float64),
                                                               ref[s2].astype(np.float64))
                elif sgd:
                    tol[th] = w.lr * dG
                else:
                    acc = ref[s1].astype(np.float64)
                    tol[s1] = 2.0 * np.abs(Gk) * dG + dG * dG
                    tol[th] = w.lr * np.minimum(2.0, 2.0 * dG / (np.sqrt(acc) + w.eps))
        for name in names:
            g = got[name].cpu().numpy()
            if sgd and name == "acc_emb":
                continue
            if sgd and name == "acc_lin" and not ftrl:
                continue
            if exact:
                assert np.array_equal(g.view(np.uint32), ref[name].view(np.uint32)), f"{what}.{name} bits"
                continue
            (close_gemm if gemm else close32)(g, ref[name], f"{what}.{name}", extra=tol.get(name))
        return ref

    # ------------------------------------------------------------------
    def step(self, batch, grads, ops=None, materialise=False, check_init=False, by_key=False,
             pooled_samples=None, dense_samples=None, head=None):
        """One full step on both sides with every intermediate compared.
        pooled_samples: compare `pooled` only on these sample indices (the dense
        per-shard pooled partial of the oracle is too large at full size).
        dense_samples: full-size first-layer workloads — the oracle's per-shard partial
        products P_s (S x B x H x F k multiply-adds) are skipped; `pooled` is compared in
        full against the unsubstituted operator, Z on these sample indices against the
        unsubstituted operator on the sub-batch; the backward is compared in full.
        head: dict(hc=constants of the fixed read-out, y=labels [B], xdense=[B][n] or None) — the upstream
        gradients are then not `grads` but what the read-out makes of each side's own forward (a closed
        loop); with resync the CUDA backward is still fed the oracle's gradients, without it its own."""
        from paper_1909_04823_b200.binding import DeviceBatch
        w = self.w
        ops = w.ops if ops is None else ops
        B, F, k, S, H = batch.batch, w.fields, w.emb_dim, w.shards, w.hidden
        dev = "cuda"
        cmp = close_gemm if self.drifted else close32
        TOL_CONTEXT[0] = f"{w.name} B={B} S={S} k={k}"
        # ---- index
        fi = self.o.find_or_insert(batch)
        db = DeviceBatch.from_synth(batch)
        self.t.find_or_insert(db, True)
        self.compare_index(batch, fi, db, by_key=by_key)
        if check_init:
            self.compare_rows(fi, db, exact=True, what="initial rows")
        # ---- forward
        op = self.o.forward_partials(ops, batch, fi, want_pooled=pooled_samples is None and dense_samples is None,
                                     want_dense=bool(ops & OP_DENSE1) and dense_samples is None)
        oa = self.o.aggregate(B, op)
        fo = self.o.forward_original(ops & ~OP_DENSE1, batch)
        sabs = fo["Sabs"]
        if dense_samples is not None and (ops & (OP_POOL | OP_DENSE1)):
            oa["pooled"] = fo["pooled"]
        xa, xl = SUMTOL_FWD * sabs[:, :k], SUMTOL_FWD * sabs[:, k]
        part_small = torch.full((S, B, k + 4), float("nan"), device=dev)
        pooled = torch.full((B, F * k), float("nan"), device=dev)
        part_pooled = torch.empty((S, B, F * k), device=dev) if materialise else None
        part_dense = torch.empty((S, B, H), device=dev) if (materialise and (ops & OP_DENSE1)) else None
        out_small = torch.full((B, k + 4), float("nan"), device=dev)
        Z = torch.full((B, max(H, 1)), float("nan"), device=dev)
        self.t.forward_partials(ops, db, part_small, pooled, part_pooled, part_dense)
        self.t.aggregate(ops, db, part_small, pooled, part_pooled, part_dense, out_small, pooled, Z)
        torch.cuda.synchronize()
        assert self.t.status() == 0
        fused_osm = None
        if not materialise:
            # the fused call (partials kept on chip) must reproduce the two-call path: bit for bit, except that
            # with pooling among the operators its aggregates come from one gather pass in another (field-wise)
            # order of addition and are held to the oracle's tolerance below
            f_small = torch.full((B, k + 4), float("nan"), device=dev)
            f_pooled = torch.full((B, F * k), float("nan"), device=dev)
            f_Z = torch.full((B, max(H, 1)), float("nan"), device=dev)
            self.t.forward_fused(ops, db, None, f_pooled, f_small, f_Z)
            torch.cuda.synchronize()
            assert self.t.status() == 0
            if (ops & (OP_LR | OP_FM)) and (ops & (OP_POOL | OP_DENSE1)):
                fused_osm = f_small.cpu().numpy()
                # ... and its shard-by-shard form (partials formed on chip in shard order) is bit-identical
                s_small = torch.full((B, k + 4), float("nan"), device=dev)
                s_pooled = torch.full((B, F * k), float("nan"), device=dev)
                s_Z = torch.full((B, max(H, 1)), float("nan"), device=dev)
                self.t.forward_fused(ops | 16, db, None, s_pooled, s_small, s_Z)
                torch.cuda.synchronize()
                assert self.t.status() == 0
                assert torch.equal(s_small.view(torch.int32), out_small.view(torch.int32)), "fused (shard order) out_small"
                assert torch.equal(s_pooled.view(torch.int32), pooled.view(torch.int32)), "fused (shard order) pooled"
            elif ops & (OP_LR | OP_FM):
                assert torch.equal(f_small.view(torch.int32), out_small.view(torch.int32)), "fused out_small"
            if ops & (OP_POOL | OP_DENSE1):
                assert torch.equal(f_pooled.view(torch.int32), pooled.view(torch.int32)), "fused pooled"
            if ops & OP_DENSE1:
                assert torch.equal(f_Z.view(torch.int32), Z.view(torch.int32)), "fused Z"
        ps = part_small.cpu().numpy()
        osm = out_small.cpu().numpy()
        AA = np.sum(oa["A"] ** 2, axis=1)
        for o_, tag in ((osm, ""), (fused_osm, "fused ")):
            if o_ is None or not (ops & (OP_LR | OP_FM)):
                continue
            if ops & OP_FM:
                cmp(o_[:, :k], oa["A"], tag + "A", extra=xa, sumabs=sabs[:, :k])
                cmp(o_[:, k + 2], oa["Q"], tag + "Q", extra=SUMTOL_FWD * oa["Q"])
                # fm2 = (<A,A> - Q)/2 subtracts two float32-rounded inputs of size <A,A>/2 and Q/2
                cmp(o_[:, k + 1], oa["fm2"], tag + "fm2",
                    extra=SUMTOL_FWD * (AA + np.abs(oa["Q"])) + np.sum(np.abs(oa["A"]) * xa, axis=1))
            else:
                assert not np.any(o_[:, :k]) and not np.any(o_[:, k + 1:k + 3]), tag + "FM outputs must be zero without FM"
            if ops & OP_LR:
                cmp(o_[:, k], oa["lr"], tag + "R_lr", extra=xl, sumabs=sabs[:, k])
            else:
                assert not np.any(o_[:, k]), tag + "R_lr must be zero without LR"
            assert not np.any(o_[:, k + 3]), "padding must be zero"
        if ops & OP_FM:
            cmp(ps[:, :, :k], op["part_small"][:, :, :k], "part_small.M1_fm", extra=xa[None], sumabs=sabs[None, :, :k])
            cmp(ps[:, :, k + 1], op["part_small"][:, :, k + 1], "part_small.M2_fm",
                extra=SUMTOL_FWD * op["part_small"][:, :, k + 1])
        if ops & OP_LR:
            cmp(ps[:, :, k], op["part_small"][:, :, k], "part_small.M1_lr", extra=xl[None], sumabs=sabs[None, :, k])
        if ops & (OP_LR | OP_FM):
            assert not np.any(ps[:, :, k + 2:]), "padding must be zero"
        if (ops & (OP_POOL | OP_DENSE1)) and pooled_samples is not None:
            sel = np.asarray(pooled_samples)
            sb = select_samples(batch, sel)
            ref_p = self.o.forward_original(ops & ~OP_DENSE1, sb)["pooled"]
            cmp(pooled[torch.from_numpy(sel).to(dev)].cpu().numpy(), ref_p, "pooled (sampled)")
        elif ops & (OP_POOL | OP_DENSE1):
            cmp(pooled.cpu().numpy(), oa["pooled"], "pooled")
            if materialise:
                cmp(part_pooled.cpu().numpy(), op["part_pooled"], "part_pooled")
        if (ops & OP_DENSE1) and dense_samples is not None:
            sel = np.asarray(dense_samples)
            ref_Z = self.o.forward_original(ops, select_samples(batch, sel))["Z"]
            close_gemm(Z[torch.from_numpy(sel).to(dev)].cpu().numpy(), ref_Z, "Z (sampled)")
        elif ops & OP_DENSE1:
            close_gemm(Z.cpu().numpy(), oa["Z"], "Z")
            if materialise:
                close_gemm(part_dense.cpu().numpy(), op["part_dense"], "part_dense")
        # ---- the read-out in place of the rest of the model: each side's gradients from its own forward
        head_out = None
        if head is not None:
            import oracle as _orc
            hc, yv, xd = head["hc"], head["y"], head.get("xdense")
            pool_term = bool(ops & OP_POOL) and not (ops & OP_DENSE1)
            oh = _orc.head(hc, oa["lr"] if ops & OP_LR else None, oa["fm2"] if ops & OP_FM else None,
                           oa["Z"] if ops & OP_DENSE1 else None, oa["pooled"] if pool_term else None, xd, yv)
            td_ = lambda a: None if a is None else torch.from_numpy(np.ascontiguousarray(a)).to(dev)
            hcd = {n: (td_(v) if isinstance(v, np.ndarray) and v.ndim else v) for n, v in hc.items()}
            h_logit = torch.full((B,), float("nan"), device=dev); h_loss = torch.full((B,), float("nan"), device=dev)
            h_gL = torch.zeros(B, device=dev); h_gF = torch.zeros(B, device=dev)
            h_gE = torch.full((B, F * k), float("nan"), device=dev) if pool_term else None
            h_gZ = torch.full((B, H), float("nan"), device=dev) if (ops & OP_DENSE1) else None
            self.t.head(ops, B, hcd, out_small, pooled, Z if (ops & OP_DENSE1) else None, td_(xd), td_(yv), h_logit, h_loss,
                        h_gL, h_gF, h_gE, h_gZ)
            torch.cuda.synchronize()
            assert self.t.status() == 0
            # the read-out sums hundreds of float32 forward results: a looser bound than the path's own
            hcmp = close_gemm if ((ops & OP_DENSE1) or self.drifted) else (lambda a, r, wh: close32(a, r, wh, rtol=1e-4, atol=1e-5))
            hcmp(h_logit.cpu().numpy(), oh["logit"], "head.logit")
            hcmp(h_loss.cpu().numpy(), oh["loss"], "head.loss")
            if ops & OP_LR:
                hcmp(h_gL.cpu().numpy() * B, oh["gL"] * B, "head.gL")
            if ops & OP_FM:
                hcmp(h_gF.cpu().numpy() * B, oh["gF"] * B, "head.gF")
            if pool_term:
                hcmp(h_gE.cpu().numpy() * B, oh["gE"] * B, "head.gE")
            if ops & OP_DENSE1:
                # a unit whose pre-activation is within rounding of zero may switch on one side only
                gz_g, gz_o = h_gZ.cpu().numpy() * B, oh["gZ"] * B
                flip = (gz_g == 0) != (gz_o == 0)
                pre = np.abs(oa["Z"] + hc["b1"][None, :].astype(np.float64))
                assert np.all(pre[flip] <= 2e-2 * np.abs(oa["Z"][flip]) + 1e-3 * np.abs(oa["Z"]).max()), "relu gate"
                hcmp(np.where(flip, gz_o, gz_g), gz_o, "head.gZ")
            f32 = lambda a: None if a is None else np.ascontiguousarray(a, dtype=np.float32)
            grads = {n: f32(oh[n]) for n in ("gL", "gF", "gE", "gZ") if oh[n] is not None}
            for n in ("gL", "gF"):
                grads.setdefault(n, np.zeros(B, np.float32))
            head_out = dict(oracle=oh, loss=float(oh["loss"].mean()), gpu_loss=float(h_loss.mean().item()))
        # ---- backward + update
        g = grads
        gdev = {n: torch.from_numpy(v).to(dev) for n, v in g.items()}
        if head is not None and not self.resync:
            gdev = {"gL": h_gL, "gF": h_gF}
            if h_gE is not None:
                gdev["gE"] = h_gE
            if h_gZ is not None:
                gdev["gZ"] = h_gZ
        gE_work = torch.empty((B, F * k), device=dev) if (ops & OP_DENSE1) else None
        before = self.o.read_rows(fi["uniq_shard"], fi["uniq_row"]) if w.lin_optimizer == synth.LIN_FTRL else None
        self.nstep += 1
        W1_pre = self.o.dense1_get()[0].astype(np.float64) if (ops & OP_DENSE1) else None
        ob = self.o.backward_update(ops, batch, fi, oa["A"].astype(np.float32),
                                    oa["pooled"].astype(np.float32) if oa["pooled"] is not None else None,
                                    g.get("gL"), g.get("gF"), g.get("gE") if (ops & OP_POOL) else None,
                                    g.get("gZ") if (ops & OP_DENSE1) else None)
        if self.resync:
            # stage-wise parity: the CUDA backward starts from the same aggregated forward
            # results as the oracle's (its own were compared above), so that differences
            # tolerated in the forward do not leak into the gradient comparison
            o32 = np.zeros((B, k + 4), dtype=np.float32)
            o32[:, :k] = oa["A"].astype(np.float32)
            out_small = torch.from_numpy(o32).to(dev)
            if oa["pooled"] is not None:
                pooled = torch.from_numpy(oa["pooled"].astype(np.float32)).to(dev)
        self.t.backward_update(ops, db, out_small, pooled, Z, gdev.get("gL"), gdev.get("gF"),
                               gdev.get("gE") if (ops & OP_POOL) else None,
                               gdev.get("gZ") if (ops & OP_DENSE1) else None, gE_work)
        torch.cuda.synchronize()
        assert self.t.status() == 0
        gemm = bool(ops & OP_DENSE1) or self.drifted
        W1o = None
        if ops & OP_DENSE1:
            # the CUDA path rounds gZ to bfloat16 before the product (2^-9 relative per term), the oracle does not:
            # where the terms of a row-times-column sum cancel, the bound is taken against their magnitudes
            extra_gE = 2.0 ** -8 * (np.abs(g["gZ"].astype(np.float64)) @ np.abs(W1_pre).T)
            if head is not None and not self.resync:
                # free-running loop: the CUDA backward was fed its own read-out gradients; where they differ from
                # the oracle's (compared above; a unit at the edge of its threshold is on on one side only) the
                # difference goes through the same product
                extra_gE = extra_gE + np.abs(gdev["gZ"].cpu().numpy().astype(np.float64) - g["gZ"].astype(np.float64)) @ np.abs(W1_pre).T
            close_gemm(gE_work.cpu().numpy(), ob["gE_total"], "gE_total", extra=extra_gE)
            W1o, accW1o = self.o.dense1_get()
            acc2W1o = self.o.dense1_get_state2() if w.optimizer == synth.OPT_ADAM else None
            # same reasoning as for the rows: a 2e-2-relative error of the weight gradient, pushed
            # through one optimizer application (Adagrad divides by sqrt(acc))
            Gk = ob["gW1"].astype(np.float64)
            dG = 2e-2 * np.abs(Gk) + 1e-3 * max(float(np.abs(Gk).max()), 1e-30)
            if w.optimizer == synth.OPT_SGD:
                extra = w.lr * dG
            elif w.optimizer == synth.OPT_ADAM:
                extra, dm, dv = self._adam_tol(Gk, dG, accW1o.astype(np.float64), acc2W1o.astype(np.float64))
                s1, s2 = self.t.dense1_get_state(want2=True)
                close_gemm(s1.cpu().numpy(), accW1o, "W1.m", extra=dm)
                close_gemm(s2.cpu().numpy(), acc2W1o, "W1.v", extra=dv)
            else:
                # G / sqrt(acc) is bounded by 1 and, for dG below |G|, moves by at most ~2 dG / sqrt(acc)
                extra = w.lr * np.minimum(2.0, 2.0 * dG / (np.sqrt(accW1o.astype(np.float64)) + w.eps))
            close_gemm(self.t.dense1_get().cpu().numpy(), W1o, "W1", extra=extra)
        ref = self.compare_rows(fi, db, gemm=gemm, what="updated rows", G=ob, before=before)
        if self.resync:
            U = fi["U"]
            td = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
            sgd = w.optimizer == synth.OPT_SGD
            ftrl = w.lin_optimizer == synth.LIN_FTRL
            self.t.write_rows(db.uniq_rows[:U], td(ref["emb"]), td(ref["lin"]),
                              None if sgd else td(ref["acc_emb"]), None if (sgd and not ftrl) else td(ref["acc_lin"]))
            if "lin2" in ref:
                self.t.write_state2(db.uniq_rows[:U], td(ref["acc2_emb"]) if "acc2_emb" in ref and w.optimizer == synth.OPT_ADAM else None,
                                    td(ref["lin2"]))
            if W1o is not None:
                self.t.dense1_set(td(W1o))
                if not sgd:
                    self.t.dense1_set_state(td(accW1o), None if acc2W1o is None else td(acc2W1o))
            torch.cuda.synchronize()
        else:
            self.drifted = True
        return dict(fi=fi, db=db, oracle_agg=oa, out_small=osm, oracle_bwd=ob, head=head_out)
