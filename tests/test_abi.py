"""CPU-side checks of the C-ABI library: it loads, exports every declared symbol, and validates arguments
on the host before touching a device."""
import ctypes
import os
import re

import pytest

from paper_2510_20787_b200 import lte

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if not fn.endswith(".h"):
            continue
        text = open(os.path.join(ROOT, "include", fn)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names |= set(re.findall(r"\b(lte_[a-z0-9_]+)\s*\(", text))
    return names


def test_library_exports_every_declared_symbol():
    L = lte.lib()
    declared = _declared()
    assert {"lte_scores", "lte_select", "lte_attn_prefill", "lte_attn_decode", "lte_attn_bwd"} <= declared
    for name in declared:
        assert hasattr(L, name), name
    assert set(lte.EXPORTS) <= declared


def test_strerror_and_sizes():
    L = lte.lib()
    assert L.lte_strerror(0) == b"ok"
    assert b"workspace" in L.lte_strerror(-3)
    s = lte.shape(128, 16, 8192, 64, 128, 128, lte.BF16)
    per = 2 * 256 * 64 * 2 + 256 * 4 + 128 * 4 + 16          # W + R = 256 rows of keys and of values
    per = (per + 255) // 256 * 256
    assert lte.lte_cache_bytes(s) == 256 + 128 * 16 * per
    c = lte.LteConv(1, 7, 1, 16, 0)
    assert lte.lte_workspace_bytes(lte.OP_BWD, s, c) > 2 * 128 * 16 * 8192 * 4
    assert lte.lte_workspace_bytes(lte.OP_SCORES, s, c) == 0


def test_host_side_validation_rejects_bad_arguments():
    L = lte.lib()
    a = ctypes.addressof
    good = lte.shape(1, 2, 128, 32, 16, 8, lte.F32)
    conv = lte.LteConv(1, 5, 1, 256, 0)
    fake = 4096          # never dereferenced: validation fails first
    assert L.lte_scores(None, a(conv), fake, fake, fake, None, None, 0, None) == -1
    assert L.lte_scores(a(good), None, fake, fake, fake, None, None, 0, None) == -1
    assert L.lte_scores(a(good), a(conv), None, fake, fake, None, None, 0, None) == -1
    assert L.lte_scores(a(good), a(conv), fake + 4, fake, fake, None, None, 0, None) == -1      # misaligned
    even = lte.LteConv(1, 4, 1, 256, 0)
    assert L.lte_scores(a(good), a(even), fake, fake, fake, None, None, 0, None) == -1
    # stacks other than the paper's (3 layers, kernel 3, dilation 2, d = 32 or 64) are unsupported
    for deep in (lte.LteConv(2, 3, 2, 256, 0), lte.LteConv(3, 5, 2, 256, 0), lte.LteConv(3, 3, 1, 256, 0)):
        assert L.lte_scores(a(good), a(deep), fake, fake, fake, None, None, 0, None) == -2
    wide = lte.shape(1, 2, 128, 128, 16, 8, lte.F32)
    assert L.lte_scores(a(wide), a(lte.LteConv(3, 3, 2, 256, 0)), fake, fake, fake, None, None, 0, None) == -2
    narrow = lte.shape(1, 2, 128, 32, 6, 8, lte.F32)          # window shorter than the stack's look-ahead + 1
    assert L.lte_scores(a(narrow), a(lte.LteConv(3, 3, 2, 256, 0)), fake, fake, fake, None, None, 0, None) == -1
    bad_d = lte.shape(1, 2, 128, 48, 16, 8, lte.F32)
    assert L.lte_scores(a(bad_d), a(conv), fake, fake, fake, None, None, 0, None) == -2
    narrow = lte.shape(1, 2, 128, 32, 3, 8, lte.F32)
    assert L.lte_scores(a(narrow), a(conv), fake, fake, fake, None, None, 0, None) == -1        # W < K
    assert L.lte_select(a(good), None, fake, fake, None, None, 0, None) == -1
    assert L.lte_attn_prefill(a(good), fake, fake, fake, fake, fake, None, fake, None, 0, None) == -1
    assert L.lte_attn_decode(a(good), a(conv), None, fake, fake, fake, fake, fake, None) == -1
    args = [a(good), a(conv)] + [fake] * 9 + [None] + [fake] * 4 + [None, 0, fake, 16, None]
    assert L.lte_attn_bwd(*args) == -3                                                         # workspace too small
    assert lte.lte_cache_bytes(lte.shape(0, 2, 1, 32, 16, 8, lte.F32)) == 0


def test_three_layer_stack_and_groups_host_side():
    """Workspace sizes and argument checks of the entry points that take the three-layer stack or grouped queries
    (no kernel is launched: validation fails first, or only sizes are asked for)."""
    L = lte.lib()
    a = ctypes.addressof
    fake = 4096
    stack = lte.LteConv(3, 3, 2, 256, 0)
    single = lte.LteConv(1, 7, 1, 256, 0)
    s = lte.shape(4, 16, 4096, 64, 128, 128, lte.BF16)
    assert lte.lte_workspace_bytes(lte.OP_SCORES, s, stack) == 16 * 194176            # the split weight image per head
    assert lte.lte_workspace_bytes(lte.OP_SCORES, lte.shape(4, 16, 4096, 64, 128, 128, lte.F32), stack) == 0
    assert lte.lte_workspace_bytes(lte.OP_SCORES, lte.shape(4, 16, 4096, 32, 128, 128, lte.BF16), stack) == 16 * 194176   # d = 32 takes the same image (zero channels)
    dec = lte.lte_workspace_bytes(lte.OP_DECODE, s, stack)                             # ring copy (k, v), its logits, the image
    assert dec >= 2 * 4 * 16 * 128 * 64 * 2 + 4 * 16 * 128 * 4 + 16 * 194176
    assert lte.lte_workspace_bytes(lte.OP_DECODE, s, single) == 0
    assert lte.lte_workspace_bytes(lte.OP_BWD, s, stack) > 16 * 129664                 # weight image + per-CTA partial gradients
    # lte_cache_score: the stack only, a window of at least 20, an aligned and large enough workspace
    assert L.lte_cache_score(a(s), a(single), fake, fake, 1 << 30, None) == -2
    assert L.lte_cache_score(a(s), a(stack), None, fake, 1 << 30, None) == -1
    assert L.lte_cache_score(a(s), a(stack), fake, None, 0, None) == -3
    assert L.lte_cache_score(a(s), a(stack), fake, fake, 16, None) == -3
    assert L.lte_cache_score(a(s), a(stack), fake, fake + 16, 1 << 30, None) == -3     # not 256-byte aligned
    short = lte.shape(4, 16, 4096, 64, 16, 8, lte.BF16)
    assert L.lte_cache_score(a(short), a(stack), fake, fake, 1 << 30, None) == -1
    assert L.lte_attn_decode(a(short), a(stack), fake, fake, fake, fake, fake, fake, None) == -1
    # the stack's backward: d = 64 and d = 32 only; negative group counts are rejected everywhere
    s128 = lte.shape(1, 2, 128, 128, 16, 8, lte.BF16)
    args = [a(s128), a(stack)] + [fake] * 9 + [None] + [fake] * 4 + [None, 0, fake, 1 << 30, None]
    assert L.lte_attn_bwd(*args) == -2
    neg = lte.shape(1, 2, 128, 64, 16, 8, lte.BF16, group=-1)
    assert L.lte_attn_prefill(a(neg), fake, fake, fake, fake, fake, fake, fake, None, 0, None) == -1
    # the shape struct ends with the group field (the binding and the header agree on the layout)
    assert ctypes.sizeof(lte.LteShape) == 11 * 4 and lte.LteShape.group.offset == 40


def test_chunked_prefill_host_side():
    """Workspace size and argument checks of lte_attn_prefill_chunk (validation fails before anything is launched)."""
    L = lte.lib()
    a = ctypes.addressof
    fake = 4096
    single = lte.LteConv(1, 7, 1, 256, 0)
    s = lte.shape(4, 16, 1024, 64, 128, 128, lte.BF16)
    ws = lte.lte_workspace_bytes(lte.OP_CHUNK, s, single)
    rows = 128 + 128 + 1024                                                   # pool + ring + chunk: the longest local sequence
    assert ws >= 2 * 64 * rows * 64 * 2 + 2 * 64 * rows * 4                   # its keys and values, two logit arrays
    assert ws % 256 == 0
    stack = lte.LteConv(3, 3, 2, 256, 0)
    assert lte.lte_workspace_bytes(lte.OP_CHUNK, s, stack) >= ws + 16 * 194176   # plus the stack's weight image
    assert lte.lte_workspace_bytes(lte.OP_CHUNK, s, None) == 0
    ok = [a(s), a(single), fake, 0, fake, fake, fake, fake, fake, fake, 1 << 40, None]
    def call(**kw):
        args = list(ok)
        for i, v in kw.items():
            args[int(i[1:])] = v
        return L.lte_attn_prefill_chunk(*args)
    assert call(_2=None) == -1                                                 # no cache
    assert call(_3=-1) == -1                                                   # negative token count
    assert call(_4=None) == -1 and call(_7=None) == -1 and call(_8=None) == -1
    assert call(_4=fake + 2) == -1                                             # misaligned q
    assert call(_9=None) == -3 and call(_10=16) == -3 and call(_9=fake + 16) == -3
    assert call(_1=a(lte.LteConv(1, 6, 1, 256, 0))) == -1                      # even tap count
    assert call(_0=a(lte.shape(4, 16, 0, 64, 128, 128, lte.BF16))) == -1       # empty chunk


def test_training_pieces_host_side():
    """Argument checks of lte_sparsity_stats (nothing is launched) and its workspace size."""
    L = lte.lib()
    a = ctypes.addressof
    fake = 4096
    s = lte.shape(8, 16, 2048, 64, 64, 64, lte.BF16)
    assert lte.lte_workspace_bytes(lte.OP_STATS, s, None) == 8 * 16 * 2 * 4
    assert L.lte_sparsity_stats(a(s), None, None, fake, fake, fake, 1 << 20, None) == -1
    assert L.lte_sparsity_stats(a(s), fake, None, None, fake, fake, 1 << 20, None) == -1
    assert L.lte_sparsity_stats(a(s), fake, None, fake, fake, None, 0, None) == -3
    assert L.lte_sparsity_stats(a(s), fake, None, fake, fake, fake, 8, None) == -3
    wide = lte.shape(1, 9000, 16, 64, 8, 4, lte.BF16)
    assert L.lte_sparsity_stats(a(wide), fake, None, fake, fake, fake, 1 << 20, None) == -2


def test_unrope_scoring_host_side():
    """lte_cache_score_unrope: both tables or none, a positive length (validation fails before anything is launched)."""
    L = lte.lib()
    a = ctypes.addressof
    fake = 4096
    stack = lte.LteConv(3, 3, 2, 256, 0)
    s = lte.shape(4, 16, 0, 64, 128, 128, lte.BF16)
    assert L.lte_cache_score_unrope(a(s), a(stack), fake, fake, None, 100, fake, 1 << 30, None) == -1
    assert L.lte_cache_score_unrope(a(s), a(stack), fake, None, fake, 100, fake, 1 << 30, None) == -1
    assert L.lte_cache_score_unrope(a(s), a(stack), fake, fake, fake, 0, fake, 1 << 30, None) == -1
    assert L.lte_cache_score_unrope(a(s), a(stack), fake, fake, fake, 100, fake, 16, None) == -3
    assert L.lte_cache_score_unrope(a(s), a(lte.LteConv(1, 7, 1, 256, 0)), fake, fake, fake, 100, fake, 1 << 30, None) == -2


def test_per_device_table_initialises_once_per_device_under_threads():
    """The launchers keep their once-per-device facts (SM count, raised shared-memory limits, symbol addresses) in a
    table indexed by device ordinal and guarded by a mutex.  Two threads that ask for the same ordinals at the same time
    (ctypes releases the interpreter lock around the calls) must see exactly one initialisation per ordinal."""
    import threading
    L = lte.lib()
    errs = []

    def worker():
        for n in range(3000):
            for dev in (0, 1, 5, 63):
                if L.lte_selftest_per_device(dev) != 1:
                    errs.append(dev)

    ts = [threading.Thread(target=worker) for _ in range(2)]
    for t in ts:
        t.start()
    for t in ts:
        t.join()
    assert not errs
    assert L.lte_selftest_per_device(64) == -1 and L.lte_selftest_per_device(-1) == -1


def test_selection_rules_host_side():
    L = lte.lib()
    s = lte.shape(1, 1, 64, 64, 8, 4, lte.BF16)
    p = ctypes.addressof(s)
    assert L.lte_select_rule(p, 7, 256, 256, 256, None, None, 0, None) == -1            # unknown rule
    assert L.lte_select_rule(p, lte.RULE_ACCUM_ATTN, None, 256, 256, None, None, 0, None) == -1   # this rule reads a score
    assert L.lte_select_rule(p, lte.RULE_UNIFORM, None, 256, None, None, None, 0, None) == -1     # cnt is required
    assert L.lte_select_rule(p, lte.RULE_LEARNED, None, 256, 256, None, None, 0, None) == -1      # lte_select's own check
    assert L.lte_attn_colsum(p, None, 256, 256, 256, 256, 256, None) == -1


def test_streaming_chunk_host_side():
    L = lte.lib()
    s = lte.shape(1, 2, 64, 64, 16, 8, lte.BF16)
    c = lte.LteConv(1, 7, 1, 256, 0)
    ps, pc = ctypes.addressof(s), ctypes.addressof(c)
    need0 = lte.lte_workspace_bytes(lte.OP_CHUNK, s, c)
    need1 = lte.lte_workspace_bytes(lte.OP_CHUNK_STREAM, s, c)
    assert need1 > need0 > 0 and need1 % 256 == 0            # the entry list and its leave times come on top
    args = (ps, pc, 256, 0, 256, 256, 256, 256, 256)
    assert L.lte_attn_prefill_chunk_ex(*args, 2, 256, need1, None) == -1          # unknown flag
    assert L.lte_attn_prefill_chunk_ex(*args, lte.CHUNK_STREAMING, 256, need0, None) == -3   # the streaming scratch is larger
    big = lte.shape(1, 2, 64, 64, 16, 5000, lte.BF16)
    assert L.lte_attn_prefill_chunk_ex(ctypes.addressof(big), pc, 256, 0, 256, 256, 256, 256, 256, lte.CHUNK_STREAMING, 256, 1 << 40, None) == -2
