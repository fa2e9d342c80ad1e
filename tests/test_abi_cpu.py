"""Host-side checks that need no GPU: the library loads, exports every symbol the public
header declares, and its pure host logic (configuration checks, workspace sizing) behaves."""
import ctypes as C
import os
import re

import pytest

from paper_2506_23431_b200 import binding as B
from paper_2506_23431_b200 import workload as W

HEADER = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "include", "pd.h")


def declared_symbols():
    text = open(HEADER).read()
    return sorted(set(re.findall(r"PD_API[^;(]*?\b(pd_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = declared_symbols()
    assert len(names) >= 20 and "pd_init" in names and "pd_step" in names and "pd_collect" in names
    lib = C.CDLL(B.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), f"libpd.so does not export {n}"
    assert set(names) == set(B.EXPORTS), "binding and header disagree on the entry points"
    assert B.version().startswith("pd-b200")


def test_config_struct_matches_header_field_order():
    text = open(HEADER).read()
    body = text[text.index("typedef struct {", text.index("PD_BUF_STATE")):text.index("} pd_config;")]
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    fields = []
    for typ, names in re.findall(r"(int32_t|float)\s+([^;]+);", body):
        fields += [(n.strip(), typ) for n in names.split(",")]
    got = [(n, "float" if t is C.c_float else "int32_t") for n, t in B.PdConfig._fields_]
    assert got == fields


@pytest.mark.parametrize("name", W.CONFIG_ORDER)
def test_workspace_bytes_of_the_five_configs(name):
    wl = W.CONFIGS[name]
    cfg = B.make_config(wl.hyper(), wl.batch)
    n = B._lib.pd_workspace_bytes(C.byref(cfg))
    e = 2 if wl.dtype == "bf16" else 4
    cross = wl.n_layers * wl.batch * wl.ctx * 2 * wl.d_model * e
    pps = -(-(wl.max_sub_len + 1) // wl.page_tokens)
    pool = wl.n_layers * wl.batch * wl.sub_max * pps * 2 * wl.d_model * wl.page_tokens * e
    assert n >= cross + pool
    assert n < 40e9                      # fits one B200 with room to spare
    cfg.pool_pages = 1
    assert B._lib.pd_workspace_bytes(C.byref(cfg)) < n


def test_invalid_configurations_are_rejected_on_the_host():
    wl = W.CONFIGS["tiny"]
    def ws(**kw):
        cfg = B.make_config(wl.hyper(), 1)
        for k, v in kw.items():
            setattr(cfg, k, v)
        return B._lib.pd_workspace_bytes(C.byref(cfg))
    assert ws() > 0
    assert ws(d_head=32) == 0
    assert ws(n_heads=3) == 0
    assert ws(sub_max=65) == 0
    assert ws(page_tokens=8) == 0
    assert ws(delta_t=0) == 0
    assert ws(dtype=7) == 0
    assert ws(sep_id=10 ** 6) == 0
    assert ws(pos_mode=3) == 0
    assert ws(kv_c_dtype=1) == 0                       # 8-bit context keys/values need the bf16 path
    assert B._lib.pd_workspace_bytes(None) == 0
    # limits of the build are told apart from bad fields, with a text
    def check(**kw):
        cfg = B.make_config(wl.hyper(), 1)
        for k, v in kw.items():
            setattr(cfg, k, v)
        why = C.c_char_p()
        return B._lib.pd_config_check(C.byref(cfg), C.byref(why)), (why.value or b"").decode()
    assert check() == (0, "")
    st, why = check(time_max=600)
    assert st == -7 and "512" in why and ws(time_max=600) == 0
    st, why = check(kv_c_dtype=1)
    assert st == -7 and "bf16" in why
    assert check(sub_max=65)[0] == -1
    # pd_init refuses null pointers and bad configs before touching CUDA
    h = C.c_void_p()
    cfg = B.make_config(wl.hyper(), 1)
    w = B.PdWeights()
    assert B._lib.pd_init(None, C.byref(w), None, 0, None, C.byref(h)) == -1
    assert B._lib.pd_init(C.byref(cfg), C.byref(w), C.c_void_p(256), 1 << 40, None, C.byref(h)) == -1  # null weights
    assert h.value is None
    assert B._lib.pd_step(None, None) == -1
    assert B._lib.pd_last_error(None) == b"null handle"


def test_rows_per_sequence_bound():
    """rows = min(sub_max, floor(max_sub_len/delta_t) + 1): a subsequence admitted at step s
    is open for at most max_sub_len + 1 steps, and admissions are delta_t apart."""
    for name in W.CONFIG_ORDER:
        wl = W.CONFIGS[name]
        fl = W.make_forced_len(wl)
        rows = min(wl.sub_max, wl.max_sub_len // wl.delta_t + 1)
        worst = 0
        for b in range(wl.batch):
            for t in range(1, wl.time_max + 1):
                n = sum(1 for i, m in enumerate(fl[b], start=1)
                        if (i - 1) * wl.delta_t + 1 <= t <= (i - 1) * wl.delta_t + 1 + m)
                worst = max(worst, n)
        assert worst <= rows
    assert min(32, 8 // 1 + 1) == 9          # keyphrase config: 9 rows per sequence, not 32


def test_pure_host_helpers_of_the_stand_alone_ops():
    """Sizing helpers that need no GPU: the projection kernel's tile plan (the number of partial sums-of-squares it
    writes = column slices x CTAs along K), scratch sizes, and their refusals."""
    lib = B._lib
    assert lib.pd_linear_sumsq_parts(1024, 1024) == 128          # 16 slices of 64 columns x 8 CTAs along K
    assert lib.pd_linear_sumsq_parts(4096, 1024) == 128
    assert lib.pd_linear_sumsq_parts(1024, 4096) > 0 and lib.pd_linear_sumsq_parts(768, 2304) > 0
    assert lib.pd_linear_sumsq_parts(96, 64) == 0 and lib.pd_linear_sumsq_parts(64, 8) == 0     # d_in % 64, d_out % 16
    assert lib.pd_linear_scratch_bytes(1024, 1024) >= 1024 * 1024 * 2 and lib.pd_linear_scratch_bytes(96, 64) == 0
    assert lib.pd_vocab_argmax_scratch_bytes(128, 32128) > 0
    assert lib.pd_cross_attention_scratch_bytes(4, 16, 8, 2) > 0 and lib.pd_cross_attention_scratch_bytes(4, 65, 8, 2) == 0
    assert lib.pd_teacher_forward_scratch_bytes(None, 100, 1) == 0
    assert lib.pd_cross_attention_static_max_bytes() == 8 << 20
