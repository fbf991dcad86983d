"""CPU-side checks of the C ABI: the library loads, exports every function that include/mkv.h
declares, validates arguments without a device, and its host bookkeeping (free lists, sequence
rows of Algorithm 1) agrees with the oracle's lifecycle model."""
import ctypes as C
import os
import random
import re

import numpy as np
import pytest

import paper_2608_23834_b200 as M
from oracle.lifecycle import LifecycleError, PoolModel

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "mkv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mkv_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_function():
    names = declared_functions()
    assert len(names) >= 25 and "mkv_decode_attention" in names and "mkv_decode_attention_static" in names
    L = M.lib()
    for n in names:
        assert hasattr(L, n), f"{n} is declared in mkv.h but not exported by libmkv.so"
    assert sorted(M.EXPORTS) == names          # the Python binding names exactly the same calls


def test_query_and_argument_validation_without_a_device():
    cfg = M.make_config(256, 4, 24, 100, 1000, np.ones(256, np.int8))
    fp8, tq3 = M.mkv_pool_query(cfg)
    assert fp8 == 100 * 4 * 32 * 256 + 256 and tq3 == 1000 * 4 * (16 * 256 + 32)
    assert M.mkv_decode_workspace_bytes(cfg, 2) >= 2 * 160 * (8 * 256 + 16) * 4
    for bad in (dict(head_dim=96), dict(n_q_heads=36), dict(n_q_heads=25), dict(fp8_pages=-1)):
        kw = dict(head_dim=256, n_kv_heads=4, n_q_heads=24, fp8_pages=1, tq3_pages=1)
        kw.update(bad)
        c = M.make_config(kw["head_dim"], kw["n_kv_heads"], kw["n_q_heads"], kw["fp8_pages"], kw["tq3_pages"],
                          np.ones(max(kw["head_dim"], 1), np.int8))
        with pytest.raises(M.MkvError) as e:
            M.mkv_pool_query(c)
        assert e.value.code == M.E_INVALID
    c = M.make_config(128, 1, 1, 1, 1, np.ones(128, np.int8))
    for bad_page in (0, 8, 24, 4112):                       # a page is 16 M tokens, M <= 256
        c.page_size = bad_page
        with pytest.raises(M.MkvError):
            M.mkv_pool_query(c)
    # pages of 1,792 tokens, 4 KV heads, d = 256: the block sizes behind the paper's byte counters (Section 5.4)
    c = M.make_config(256, 4, 24, 18, 47, np.ones(256, np.int8), page_tokens=1792)
    fp8, tq3 = M.mkv_pool_query(c)
    assert fp8 - 256 + tq3 == 131_610_624
    # device calls on a bookkeeping-only pool are refused, not attempted
    hp = M.HostPool(128, 2, 8, 4, 4)
    L = M.lib()
    assert L.mkv_append(hp.handle, None, None, None, 1, None) == M.E_INVALID
    assert L.mkv_decode_attention(hp.handle, None, None, None, None, 1, 1, 1.0, None, None, None, 0, None) == M.E_INVALID
    assert L.mkv_pool_status(hp.handle, None) == M.E_INVALID
    assert L.mkv_page_read_raw(hp.handle, 0, 0, None, None) == M.E_INVALID
    hp.close()


def test_free_lists_hand_out_ids_in_order_and_reject_misuse():
    hp = M.HostPool(128, 2, 8, 5, 3)
    assert hp.page_alloc(M.FMT_FP8, 3).tolist() == [0, 1, 2]
    assert hp.page_alloc(M.FMT_TQ3, 3).tolist() == [0, 1, 2]
    with pytest.raises(M.MkvError) as e:
        hp.page_alloc(M.FMT_FP8, 3)                     # only 2 left: all-or-nothing
    assert e.value.code == M.E_OOM_FP8
    with pytest.raises(M.MkvError) as e:
        hp.page_alloc(M.FMT_TQ3, 1)
    assert e.value.code == M.E_OOM_TQ3
    hp.page_free(M.FMT_FP8, [1])
    assert hp.page_alloc(M.FMT_FP8, 1).tolist() == [1]   # a freed id is reused first
    for ids, code in (([1, 1], M.E_STATE), ([7], M.E_BOUNDS), ([-1], M.E_BOUNDS), ([4], M.E_STATE)):
        with pytest.raises(M.MkvError) as e:
            hp.page_free(M.FMT_FP8, ids)
        assert e.value.code == code
    st = hp.stats()
    assert (st.fp8_pages_used, st.tq3_pages_used) == (3, 3)
    assert st.fp8_bytes_used == 3 * 2 * 32 * 128 and st.tq3_bytes_used == 3 * 2 * (16 * 128 + 32)
    assert st.bf16_bytes_equivalent == 6 * 2 * 16 * 128 * 4
    hp.close()


CODES = {"MKV_E_OOM_FP8": M.E_OOM_FP8, "MKV_E_OOM_TQ3": M.E_OOM_TQ3, "MKV_E_STATE": M.E_STATE, "MKV_E_BOUNDS": M.E_BOUNDS}


@pytest.mark.parametrize("page_tokens", [16, 48])
def test_sequence_bookkeeping_agrees_with_the_lifecycle_model_on_a_random_walk(page_tokens):
    """Same transitions on the library's mkv_seq_* and on the oracle's model of Algorithm 1: same
    rows (tags and physical ids), same failures, same pool occupancy, after every step (pages of 16
    tokens, and pages of three 16-token tiles)."""
    rnd = random.Random(page_tokens)
    hp = M.HostPool(128, 2, 8, 24, 24, page_tokens=page_tokens)
    model = PoolModel(24, 24, page_tokens)
    seqs = []          # (library Seq, model SeqModel)
    for step in range(3000):
        r = rnd.random()
        if r < 0.03 or not seqs:
            seqs.append((M.Seq(hp), model.new_seq()))
            continue
        i = rnd.randrange(len(seqs))
        s, m = seqs[i]
        n_pages = len(m.pages)
        lp = rnd.randrange(n_pages + 1) if n_pages else 0       # sometimes out of range
        if r < 0.70:
            op = ("append",)
        elif r < 0.82:
            op = ("demote", lp)
        elif r < 0.86:
            op = ("promote", lp)
        elif r < 0.90:
            op = ("protect", lp, rnd.random() < 0.7)
        elif r < 0.94:
            op = ("age", rnd.choice([16, 40, 100]) * page_tokens // 16)
        elif r < 0.97:
            # the stream point of a planned conversion has passed: release one retiring source of this request
            mine = sorted(k for k, h in model.retiring.items() if h == m.handle)
            op = ("release",) + (rnd.choice(mine) if mine and rnd.random() < 0.9 else (rnd.randrange(2), rnd.randrange(26)))
        else:
            op = ("finish",)
        got = want = None
        try:
            if op[0] == "append":
                want = m.append()
            elif op[0] == "demote":
                want = m.demote(op[1])
            elif op[0] == "promote":
                want = m.promote(op[1])
            elif op[0] == "protect":
                want = m.protect(op[1]) if op[2] else m.unprotect(op[1])
            elif op[0] == "age":
                want = m.age(op[1])
            elif op[0] == "release":
                want = m.release(op[1], op[2])
            else:
                m.finish()
        except LifecycleError as e:
            want = ("error", CODES[e.code])
        try:
            if op[0] == "append":
                got = s.append()
            elif op[0] == "demote":
                got = s.demote(op[1])
            elif op[0] == "promote":
                got = s.promote(op[1])
            elif op[0] == "protect":
                got = s.protect(op[1], op[2])
            elif op[0] == "age":
                got = s.age(op[1])
            elif op[0] == "release":
                got = s.release(op[1], op[2])
            else:
                s.finish()
        except M.MkvError as e:
            got = ("error", e.code)
        if op[0] == "age" and isinstance(want, tuple) and want[0] == "error":
            # the model demotes page by page and stops at the first failure; the library plans the whole
            # batch or nothing: both report the exhausted arena
            assert got == want
            seqs.pop(i)            # states may differ after a partial batch: retire the pair
            try:
                m.finish()
            except LifecycleError:
                pass
            s.finish()
            continue
        assert got == want, (step, op, got, want)
        if op[0] == "finish":
            seqs.pop(i)
            continue
        ids, tags = s.row()
        assert [(int(t), int(p)) for t, p in zip(tags, ids)] == m.pages
        assert s.len() == (m.len, len(m.pages))
        st = hp.stats()
        used, _ = model.stats()
        assert (st.fp8_pages_used, st.tq3_pages_used) == (used[0], used[1])
        model.check_invariants()
    hp.close()
