"""The C-ABI library loads without a GPU, exports every symbol the header declares, and rejects
bad arguments on the host before touching CUDA."""
import ctypes
import os
import re

import pytest

from paper_2505_20334_b200 import build as laq_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def binding():
    laq_build.build_liblaq()
    from paper_2505_20334_b200 import binding as b
    return b


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "laq.h")).read()
    return sorted(set(re.findall(r"LAQ_API[^;(]*?\b(laq_\w+)\s*\(", text)))


def test_header_symbols_are_exported(binding):
    names = declared_symbols()
    assert len(names) >= 10 and "laq_evict" in names
    raw = ctypes.CDLL(binding.LIB_PATH)
    for n in names:
        assert hasattr(raw, n), f"{n} declared in laq.h but not exported"
    assert set(names) == set(binding.EXPORTS)


def test_struct_layout_and_version(binding):
    assert ctypes.sizeof(binding.LaqParams) == 18 * 4 + 16 * 8 + 8
    assert binding.LaqParams.q_stride_layer.offset == 72
    assert binding.laq_version() >= 100
    assert binding.status_string(0) == "ok"
    assert "argument" in binding.status_string(binding.LAQ_ERR_INVALID_ARG)


def test_dense_strides_and_workspace(binding):
    p = binding.make_params(2, 3, 8, 2, 128, 1000, 4, 4, 7, 64)
    assert (p.q_stride_pos, p.q_stride_head, p.q_stride_batch, p.q_stride_layer) == (
        128, 4 * 128, 8 * 4 * 128, 3 * 8 * 4 * 128)
    assert (p.k_stride_pos, p.k_stride_head, p.k_stride_batch) == (128, 1000 * 128, 2 * 1000 * 128)
    assert (p.o_stride_head, p.o_stride_layer) == (64 * 128, 3 * 2 * 64 * 128)
    n = binding.laq_workspace_bytes(p)
    assert n > 2 * 3 * 2 * 1000 * 4 and n % 256 == 0
    # config 5 pool: offsets beyond 2^32 bytes must not overflow
    big = binding.make_params(80, 1, 64, 8, 128, 65536, 32, 32, 7, 2048)
    assert big.k_stride_layer * 80 * 2 > 2 ** 32
    assert binding.laq_workspace_bytes(big) > 80 * 8 * 65536 * 4


@pytest.mark.parametrize("kw", [
    dict(n_q_heads=7),            # not a multiple of n_kv_heads
    dict(budget=1000),            # B >= L
    dict(budget=4),               # B <= R
    dict(pool_kernel=4),          # even kernel
    dict(keep_tail=-1),
    dict(prompt_len=0),
    dict(softmax_scale=float("nan")),
])
def test_invalid_params_rejected_on_host(binding, kw):
    args = dict(n_layers=1, batch=1, n_q_heads=8, n_kv_heads=2, head_dim=128, prompt_len=1000,
                window_len=4, keep_tail=4, pool_kernel=7, budget=64)
    args.update(kw)
    p = binding.make_params(**args)
    assert binding.laq_workspace_bytes(p) == 0
    fake = ctypes.c_void_p(4096)
    st = binding.lib.laq_evict(ctypes.byref(p), fake, fake, fake, fake, fake, fake, None, fake,
                               1 << 40, None)
    assert st == binding.LAQ_ERR_INVALID_ARG


def test_unsupported_and_pointer_checks(binding):
    p = binding.make_params(1, 1, 8, 2, 100, 1000, 4, 4, 7, 64)   # head_dim not a multiple of 8
    fake = ctypes.c_void_p(4096)
    st = binding.lib.laq_evict(ctypes.byref(p), fake, fake, fake, fake, fake, fake, None, fake,
                               1 << 40, None)
    assert st == binding.LAQ_ERR_UNSUPPORTED
    p = binding.make_params(1, 1, 64, 1, 128, 1000, 8, 8, 7, 64)  # G*W = 512 rows
    assert binding.lib.laq_score(ctypes.byref(p), fake, fake, fake, fake, 1 << 40, None) == \
        binding.LAQ_ERR_UNSUPPORTED
    p = binding.make_params(1, 1, 8, 2, 128, 1000, 4, 4, 7, 64)
    odd = ctypes.c_void_p(4096 + 8)
    assert binding.lib.laq_score(ctypes.byref(p), None, fake, fake, fake, 1 << 40, None) == \
        binding.LAQ_ERR_INVALID_ARG
    assert binding.lib.laq_score(ctypes.byref(p), odd, fake, fake, fake, 1 << 40, None) == \
        binding.LAQ_ERR_INVALID_ARG
    assert binding.lib.laq_score(ctypes.byref(p), fake, fake, fake, fake, 16, None) == \
        binding.LAQ_ERR_WORKSPACE
    assert binding.lib.laq_score(ctypes.byref(p), fake, fake, fake, None, 0, None) == \
        binding.LAQ_ERR_WORKSPACE
    p.k_stride_pos = 132  # not a multiple of 8 elements
    assert binding.lib.laq_score(ctypes.byref(p), fake, fake, fake, fake, 1 << 40, None) == \
        binding.LAQ_ERR_INVALID_ARG
    p = binding.make_params(1, 1, 8, 2, 128, 1000, 4, 4, 7, 64)
    assert binding.lib.laq_select(ctypes.byref(p), None, fake, None) == binding.LAQ_ERR_INVALID_ARG
    assert binding.lib.laq_compact(ctypes.byref(p), fake, fake, None, fake, fake, None) == \
        binding.LAQ_ERR_INVALID_ARG


def test_seq_lens_are_validated_on_host(binding):
    p = binding.make_params(1, 3, 8, 2, 128, 1000, 4, 4, 7, 64)
    base = binding.laq_workspace_bytes(p)
    p.set_seq_lens([1000, 65, 500])
    assert binding.laq_workspace_bytes(p) == base          # lengths do not change the workspace
    for bad in ([1000, 64, 500],      # a prompt no longer than the budget
                [1001, 500, 500],     # longer than the allocated length
                [1000, 500, -3]):
        p.set_seq_lens(bad)
        assert binding.laq_workspace_bytes(p) == 0
    with pytest.raises(ValueError):
        p.set_seq_lens([1000, 500])   # one length per batch item
    p.set_seq_lens(None)
    assert binding.laq_workspace_bytes(p) == base
    big = binding.make_params(1, 513, 8, 2, 128, 1000, 4, 4, 7, 64)
    big.set_seq_lens([1000] * 513)    # more prompts than LAQ_MAX_RAGGED_BATCH
    fake = ctypes.c_void_p(4096)
    assert binding.lib.laq_score(ctypes.byref(big), fake, fake, fake, fake, 1 << 40, None) == \
        binding.LAQ_ERR_UNSUPPORTED


def test_layer_budget_pool_size_and_validation_on_the_host(binding):
    p = binding.make_params(3, 2, 8, 2, 128, 1000, 4, 4, 7, 90)
    assert binding.laq_layers_pool_entries(p, [90, 40, 64]) == 2 * 2 * (90 + 40 + 64)
    assert binding.laq_layers_pool_entries(p, [80, 40, 64]) == 0      # p.budget must be the largest
    assert binding.laq_layers_pool_entries(p, [90, 4, 64]) == 0       # a budget must exceed the tail
    assert binding.laq_layers_pool_entries(p, [90, 1000, 64]) == 0    # and stay below the prompt length
    p.group_mode = binding.LAQ_GROUP_PER_HEAD                         # one row of entries per query head
    assert binding.laq_layers_pool_entries(p, [90, 40, 64]) == 2 * 8 * (90 + 40 + 64)
    p.set_seq_lens([1000, 60])
    assert binding.laq_layers_pool_entries(p, [90, 40, 64]) == 0      # a budget reaches a prompt's length


def test_group_mode_and_streaming_arguments_are_checked_on_the_host(binding):
    p = binding.make_params(1, 1, 8, 2, 128, 1000, 4, 4, 7, 90)
    n = binding.laq_workspace_bytes(p)
    p.group_mode = binding.LAQ_GROUP_MAX
    assert binding.laq_workspace_bytes(p) > n          # per-head column sums need room
    p.group_mode = 3
    assert binding.laq_workspace_bytes(p) == 0
    p.group_mode = binding.LAQ_GROUP_PER_HEAD
    p.score_mode = binding.LAQ_SCORE_RAW
    assert binding.laq_workspace_bytes(p) == 0         # unsupported together
    p.group_mode, p.score_mode, p.reserved0 = 0, 0, 1
    assert binding.laq_workspace_bytes(p) == 0
    p.reserved0 = 0
    for n_sink in (-1, 91):
        st = binding.lib.laq_streaming_indices(ctypes.byref(p), n_sink, ctypes.c_void_p(16), None)
        assert st == binding.LAQ_ERR_INVALID_ARG
    assert binding.lib.laq_streaming_indices(ctypes.byref(p), 4, None, None) == binding.LAQ_ERR_INVALID_ARG
