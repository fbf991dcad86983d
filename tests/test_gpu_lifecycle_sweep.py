"""Lifecycle sweep cell (config 4 shape, scaled): every transition goes through the library --
mkv_seq_* plans, mkv_append / mkv_demote / mkv_set_anchor kernels, mkv_decode_attention -- and is
mirrored by the oracle (lifecycle model + codecs + fp64 attention).  Packed pages and tables must
agree bit for bit, attention within the tolerance."""
import numpy as np
import pytest
import torch

import mkv_workloads as W
import oracle
import paper_2608_23834_b200 as M
from _gpu_util import bf16_tensor, check_close
from oracle.lifecycle import FMT_FP8, FMT_TQ3, PoolModel, STALE

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("frac,ctx,batch,T", [(0.5, 512, 2, 16), (0.95, 320, 3, 16), (0.0, 256, 2, 16), (0.5, 12 * 48, 2, 48)])
def test_append_demote_decode_cell(frac, ctx, batch, T):
    """T: tokens per page (16, or three 16-token tiles with one value scale/zero set per page)."""
    spec = W.config(4, batch=batch, ctx=ctx, stale_fraction=frac, n_kv_heads=2, page_tokens=T)
    d, hkv, hq = spec.head_dim, spec.n_kv_heads, spec.n_q_heads
    Mt = T // 16
    n_pages = ctx // T
    cap = batch * (n_pages + 2)
    sigma = W.rotation_signs(spec)
    pool = M.Pool(d, hkv, hq, cap, cap, sigma, max_batch=batch, page_tokens=T)
    model = PoolModel(cap, cap, T)
    fp8 = np.zeros((cap, hkv, oracle.fp8_block_bytes(d, Mt)), np.uint8)          # the oracle's own arenas
    tq3 = np.zeros((cap, hkv, oracle.tq3_block_bytes(d, Mt)), np.uint8)
    seqs = [M.Seq(pool) for _ in range(batch)]
    mods = [model.new_seq() for _ in range(batch)]
    max_pages = n_pages + 2
    bt = torch.full((batch, max_pages), -1, dtype=torch.int32, device="cuda:0")
    tags = torch.zeros((batch, max_pages), dtype=torch.uint8, device="cuda:0")

    def append_tokens(k_bits, v_bits):
        """k_bits, v_bits: [n][batch][hkv][d]; request-major interleaving of one token each per call."""
        slots = []
        for t in range(k_bits.shape[0]):
            for b in range(batch):
                pid, sl, opened = seqs[b].append()
                assert (pid, sl, opened) == mods[b].append()
                if opened:
                    bt[b, len(mods[b].pages) - 1] = pid       # publish the new Recent page
                slots.append(pid * T + sl)
                kf, vf = oracle.bf16_bits_to_f32(k_bits[t, b]), oracle.bf16_bits_to_f32(v_bits[t, b])
                for h in range(hkv):
                    rec = fp8[pid, h, (sl // 16) * 32 * d:(sl // 16 + 1) * 32 * d]     # the 16-token tile of the slot
                    s16 = sl % 16
                    rec[s16 * d:(s16 + 1) * d] = [oracle.e4m3_encode(x) for x in kf[h]]
                    rec[16 * d + s16:32 * d:16] = [oracle.e4m3_encode(x) for x in vf[h]]
        kk = bf16_tensor(k_bits.reshape(-1, hkv, d))
        vv = bf16_tensor(v_bits.reshape(-1, hkv, d))
        pool.append(kk, vv, torch.tensor(slots, dtype=torch.int32, device="cuda:0"))

    def demote(pairs):
        """pairs: list of (b, logical page, src, dst) already planned on both sides."""
        if not pairs:
            return
        for b, lp, s, t in pairs:
            for h in range(hkv):
                tq3[t, h] = oracle.demote_block(fp8[s, h], d, Mt, sigma)
        src = torch.tensor([p[2] for p in pairs], dtype=torch.int32, device="cuda:0")
        dst = torch.tensor([p[3] for p in pairs], dtype=torch.int32, device="cuda:0")
        ent = torch.tensor([p[0] * max_pages + p[1] for p in pairs], dtype=torch.int64, device="cuda:0")
        pool.demote(src, dst, bt, tags, ent)
        # everything runs on one stream: once the conversion is enqueued, later writers of the sources are ordered
        # after it and after every earlier reader, so the retiring sources can go back to their free list
        for b, lp, s, t in pairs:
            seqs[b].release(M.FMT_FP8, s)
            mods[b].release(FMT_FP8, s)

    # ---- bring the cell to its starting state: ctx tokens, oldest floor(f*P) pages Stale ----
    rng = np.random.default_rng(4)
    k0 = W.f32_to_bf16_bits(rng.standard_normal((ctx, batch, hkv, d)).astype(np.float32))
    v0 = W.f32_to_bf16_bits(rng.standard_normal((ctx, batch, hkv, d)).astype(np.float32))
    append_tokens(k0, v0)
    pairs = []
    for b in range(batch):
        for lp in range(int(np.floor(frac * n_pages))):
            s, t = seqs[b].demote(lp)
            assert (s, t) == mods[b].demote(lp)
            pairs.append((b, lp, s, t))
    demote(pairs)

    # ---- the cell: append one token, demote the page leaving the Recent window, protect one, decode ----
    k1, v1 = W.new_token_kv(spec, 0)
    append_tokens(k1[None], v1[None])
    recent = max(T, ctx - int(np.floor(frac * n_pages)) * T - T)   # the window shrinks by one page
    pairs = []
    for b in range(batch):
        moved = seqs[b].age(recent)
        assert moved == mods[b].age(recent)
        pairs += [(b,) + m for m in moved]
    demote(pairs)
    if frac == 0.5:
        assert len(pairs) == batch
    for b in range(batch):                                          # protect the newest full page
        lp = n_pages - 1
        seqs[b].protect(lp, True)
        mods[b].protect(lp)
        pool.set_anchor(tags, b * max_pages + lp, True)
    torch.cuda.synchronize()
    assert pool.status() == M.OK
    model.check_invariants()

    # tables on the device equal the host rows of both sides
    bt_h, tg_h = bt.cpu().numpy(), tags.cpu().numpy()
    for b in range(batch):
        ids, tg = seqs[b].row()
        n = len(ids)
        assert [(int(t), int(p)) for t, p in zip(tg, ids)] == mods[b].pages
        assert np.array_equal(bt_h[b, :n], ids) and np.array_equal(tg_h[b, :n], tg)
    # every live page is bit-identical to the oracle's
    for b in range(batch):
        for tag, pid in mods[b].pages:
            if tag == STALE:
                assert np.array_equal(pool.page_read_raw(M.FMT_TQ3, pid).reshape(hkv, -1), tq3[pid])
            else:
                assert np.array_equal(pool.page_read_raw(M.FMT_FP8, pid).reshape(hkv, -1), fp8[pid])
    st = pool.stats()
    used, _ = model.stats()
    assert (st.fp8_pages_used, st.tq3_pages_used) == (used[0], used[1])

    lens = np.array([m.len for m in mods], np.int32)
    q_bits = W.query(spec)
    ref, ref_lse = oracle.decode_attention(fp8, tq3, d, hkv, spec.group, sigma, q_bits, bt_h, tg_h, lens, spec.scale,
                                           page_tokens=T)
    for variant in (M.DECODE_TENSOR, M.DECODE_SCALAR):
        pool.set_decode_variant(variant)
        out = pool.decode_attention(bf16_tensor(q_bits), bt, tags, torch.from_numpy(lens).cuda(), spec.scale)
        torch.cuda.synchronize()
        assert pool.status() == M.OK
        check_close(out.cpu().numpy(), ref, f"cell f={frac} variant={variant}")
    # ---- Promote (Stale -> Anchor through a new FP8 page) the oldest Stale page of every request, decode again
    pairs = []
    for b in range(batch):
        stale = [lp for lp, (tag, _) in enumerate(mods[b].pages) if tag == STALE]
        if stale:
            s_id, t_id = seqs[b].promote(stale[0])
            assert (s_id, t_id) == mods[b].promote(stale[0])
            pairs.append((b, stale[0], s_id, t_id))
    if pairs:
        for b, lp, s_id, t_id in pairs:
            for h in range(hkv):
                fp8[t_id, h] = oracle.promote_block(tq3[s_id, h], d, Mt, sigma)
        src = torch.tensor([p[2] for p in pairs], dtype=torch.int32, device="cuda:0")
        dst = torch.tensor([p[3] for p in pairs], dtype=torch.int32, device="cuda:0")
        ent = torch.tensor([p[0] * max_pages + p[1] for p in pairs], dtype=torch.int64, device="cuda:0")
        pool.promote(src, dst, bt, tags, ent)
        torch.cuda.synchronize()
        assert pool.status() == M.OK
        # the Stale sources are retiring (counted as used, handed to nobody) until they are released
        st, (used, _) = pool.stats(), model.stats()
        assert (st.fp8_pages_used, st.tq3_pages_used) == (used[0], used[1])
        for b_, lp_, s_id, t_id in pairs:
            seqs[b_].release(M.FMT_TQ3, s_id)
            mods[b_].release(FMT_TQ3, s_id)
        model.check_invariants()
        assert pool.stats().tq3_pages_used == st.tq3_pages_used - len(pairs)
        bt_h, tg_h = bt.cpu().numpy(), tags.cpu().numpy()
        for b, lp, s_id, t_id in pairs:
            assert bt_h[b, lp] == t_id and tg_h[b, lp] == M.TAG_ANCHOR
            assert np.array_equal(pool.page_read_raw(M.FMT_FP8, t_id).reshape(hkv, -1), fp8[t_id])
        ref, _ = oracle.decode_attention(fp8, tq3, d, hkv, spec.group, sigma, q_bits, bt_h, tg_h, lens, spec.scale,
                                         page_tokens=T)
        pool.set_decode_variant(M.DECODE_TENSOR)
        out = pool.decode_attention(bf16_tensor(q_bits), bt, tags, torch.from_numpy(lens).cuda(), spec.scale)
        check_close(out.cpu().numpy(), ref, f"cell f={frac} after promote")
        model.check_invariants()
    for s in seqs:
        s.finish()
    assert pool.stats().fp8_pages_used == 0 and pool.stats().tq3_pages_used == 0
