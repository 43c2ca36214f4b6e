"""Host-side checks of the C boundary that need no GPU: exported symbols, budgets, sizes, validation."""
import ctypes
import glob
import os
import re
import subprocess
import sys

import pytest

import oracle
import paper_2406_02069_b200 as pkv
from paper_2406_02069_b200 import binding, workloads

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    names = set()
    for path in glob.glob(os.path.join(ROOT, "include", "*.h")):
        text = re.sub(r"/\*.*?\*/", "", open(path).read(), flags=re.S)
        names.update(re.findall(r"\b(pyramidkv_\w+)\s*\(", text))
    return sorted(names)


def test_library_exports_every_declared_symbol():
    lib = ctypes.CDLL(pkv.library_path())
    names = declared_functions()
    assert len(names) >= 9
    for name in names:
        assert hasattr(lib, name), name
    assert set(binding.EXPORTS) <= set(names)


@pytest.mark.parametrize("m,B,alpha,beta", [
    (2, 64, 8, 20.0), (32, 128, 32, 20.0), (32, 512, 32, 20.0), (80, 128, 32, 20.0), (32, 64, 32, 20.0),
    (32, 2048, 32, 20.0), (32, 64, 8, 14.0), (7, 33, 5, 3.5), (3, 1000, 48, 1.0), (1, 77, 8, 20.0),
    (5, 8, 8, 20.0), (600, 4096, 16, 17.25),
])
def test_budgets_match_oracle(m, B, alpha, beta):
    cfg = pkv.make_config(num_layers=m, num_q_heads=8, num_kv_heads=2, head_dim=128, window=alpha, pool_kernel=7,
                          dtype="bf16", avg_budget=B, beta=beta)
    got = pkv.layer_budgets(cfg)
    assert got == oracle.layer_budgets(m, B, alpha, beta)
    assert sum(got) == m * (B - alpha)
    for n in (alpha + 1, B - 1, B, B + 1, 10 * B + 3):
        if n < alpha + 1:
            continue
        for kl in (got[0], got[-1]):
            assert pkv.kept_count(cfg, kl, n) == oracle.kept_count(B, alpha, kl, n)


@pytest.mark.parametrize("m,B,alpha,beta", [
    (2, 64, 8, 20.0), (32, 128, 32, 20.0), (32, 512, 32, 20.0), (80, 128, 32, 20.0), (32, 64, 8, 20.0),
    (32, 2048, 32, 20.0), (32, 64, 8, 14.0), (7, 33, 5, 3.5), (3, 1000, 48, 1.0), (1, 77, 8, 20.0),
    (5, 8, 8, 20.0), (600, 4096, 16, 17.25), (3, 78, 8, 7.0), (4, 23, 8, 3.75), (16, 300, 16, 5.25),
])
def test_geometric_budgets_match_oracle(m, B, alpha, beta):
    cfg = pkv.make_config(num_layers=m, num_q_heads=8, num_kv_heads=2, head_dim=128, window=alpha, pool_kernel=7,
                          dtype="bf16", avg_budget=B, beta=beta, schedule="geometric")
    got = pkv.layer_budgets(cfg)
    assert got == oracle.layer_budgets(m, B, alpha, beta, schedule="geometric")
    assert sum(got) == m * (B - alpha) and all(a >= b for a, b in zip(got, got[1:]))


def test_invalid_configs_are_rejected_on_the_host():
    good = dict(num_layers=4, num_q_heads=8, num_kv_heads=2, head_dim=128, window=8, pool_kernel=7, dtype="bf16",
                avg_budget=64, beta=20.0)
    for bad in (dict(num_layers=0), dict(num_q_heads=7), dict(window=0), dict(avg_budget=4), dict(pool_kernel=4),
                dict(beta=0.5), dict(beta=float("nan"))):
        cfg = pkv.make_config(**{**good, **bad})
        with pytest.raises(pkv.PkvError) as e:
            pkv.layer_budgets(cfg)
        assert e.value.status == binding.PKV_ERR_INVALID_ARG
        assert pkv.workspace_bytes(cfg, 1, 1024) == 0
    cfg = pkv.make_config(**good)
    with pytest.raises(pkv.PkvError):
        pkv.kept_count(cfg, 5, 8)            # shorter than window + 1
    with pytest.raises(pkv.PkvError):
        pkv.kept_count(cfg, -1, 100)


_REFUSALS = r'''
import ctypes
import paper_2406_02069_b200 as pkv
from paper_2406_02069_b200 import binding

cfg = pkv.make_config(num_layers=4, num_q_heads=8, num_kv_heads=2, head_dim=128, window=8, pool_kernel=7,
                      dtype="bf16", avg_budget=64)
lib = binding._lib
null_t = binding.PkvTensor(None, 0, 0, 0)
lens = (ctypes.c_int32 * 1)(100)
st = lib.pyramidkv_score_window(ctypes.byref(cfg), null_t, null_t, lens, 1, None, 128, None, 0, None)
assert st == binding.PKV_ERR_INVALID_ARG
st = lib.pyramidkv_select_topk(ctypes.byref(cfg), None, 128, lens, 1, 4, None, None, 0, None)
assert st == binding.PKV_ERR_INVALID_ARG
fake = binding.PkvTensor(4096, 1 << 20, 1 << 16, 128)       # plausible but never dereferenced
short = (ctypes.c_int32 * 1)(8)
st = lib.pyramidkv_score_window(ctypes.byref(cfg), fake, fake, short, 1, 4096, 128, 4096, 1 << 30, None)
assert st == binding.PKV_ERR_INVALID_ARG                     # n < alpha + 1
many = (ctypes.c_int32 * 65)(*([100] * 65))
st = lib.pyramidkv_score_window(ctypes.byref(cfg), fake, fake, many, 65, 4096, 128, 4096, 1 << 30, None)
assert st == binding.PKV_ERR_UNSUPPORTED
st = lib.pyramidkv_score_window(ctypes.byref(cfg), fake, fake, lens, 1, 4096, 128, 4096, 16, None)
assert st == binding.PKV_ERR_WORKSPACE                       # workspace too small
st = lib.pyramidkv_score_window(ctypes.byref(cfg), fake, fake, lens, 1, 4096, 128, 4097, 1 << 30, None)
assert st == binding.PKV_ERR_WORKSPACE                       # misaligned
st = lib.pyramidkv_score_window(ctypes.byref(cfg), fake, fake, lens, 1, 4096, 16, 4096, 1 << 30, None)
assert st == binding.PKV_ERR_INVALID_ARG                     # ld_scores < prefix
odd = binding.PkvTensor(4098, 1 << 20, 1 << 16, 128)
st = lib.pyramidkv_score_window(ctypes.byref(cfg), odd, fake, lens, 1, 4096, 128, 4096, 1 << 30, None)
assert st == binding.PKV_ERR_INVALID_ARG                     # pointer not 16-byte aligned
two = (ctypes.c_int32 * 2)(100, 100)
for view in (binding.PkvTensor(4096, 0, 1 << 16, 128), binding.PkvTensor(4096, 1 << 20, 0, 128),
             binding.PkvTensor(4096, 1 << 20, -(1 << 16), 128)):        # broadcast / reversed views
    st = lib.pyramidkv_score_window(ctypes.byref(cfg), fake, view, two, 2, 4096, 128, 4096, 1 << 30, None)
    assert st == binding.PKV_ERR_INVALID_ARG
bad = pkv.make_config(num_layers=4, num_q_heads=8, num_kv_heads=2, head_dim=96, window=8, pool_kernel=7,
                      dtype="bf16", avg_budget=64)
st = lib.pyramidkv_score_window(ctypes.byref(bad), fake, fake, lens, 1, 4096, 128, 4096, 1 << 30, None)
assert st == binding.PKV_ERR_UNSUPPORTED
for field, value in (("dtype", 3), ("pool_kind", 2)):           # codes past fp16 / the mean pool are not built
    odd_cfg = pkv.make_config(num_layers=4, num_q_heads=8, num_kv_heads=2, head_dim=128, window=8, pool_kernel=7,
                              dtype="fp16", avg_budget=64, pool_kind=1)
    setattr(odd_cfg, field, value)
    st = lib.pyramidkv_score_window(ctypes.byref(odd_cfg), fake, fake, lens, 1, 4096, 128, 4096, 1 << 30, None)
    assert st == binding.PKV_ERR_UNSUPPORTED
sched = pkv.make_config(num_layers=4, num_q_heads=8, num_kv_heads=2, head_dim=128, window=8, pool_kernel=7,
                        dtype="bf16", avg_budget=64)
sched.schedule = 7                                              # no such schedule
st = lib.pyramidkv_score_window(ctypes.byref(sched), fake, fake, lens, 1, 4096, 128, 4096, 1 << 30, None)
assert st == binding.PKV_ERR_INVALID_ARG
assert pkv.strerror(binding.PKV_ERR_WORKSPACE).startswith("workspace")
print("refusals ok")
'''


def test_validation_happens_before_any_device_work():
    """Null pointers, short sequences, oversize batches, broadcast views ... are refused on the host.  The calls
    carry invented device pointers, so they run in a child process that sees no GPU: a check that came too late
    could then reach no kernel launch, whatever machine the suite runs on."""
    env = dict(os.environ, CUDA_VISIBLE_DEVICES="")
    out = subprocess.run([sys.executable, "-c", _REFUSALS], cwd=ROOT, env=env, capture_output=True, text=True,
                         timeout=600)
    assert out.returncode == 0 and "refusals ok" in out.stdout, out.stdout[-2000:] + out.stderr[-4000:]


def test_workspace_grows_with_the_problem():
    cfg = pkv.config_of(workloads.LLAMA3_70B)
    a = pkv.workspace_bytes(cfg, 1, 4096)
    b = pkv.workspace_bytes(cfg, 1, 131072)
    c = pkv.workspace_bytes(cfg, 4, 131072)
    assert 0 < a < b < c and a % 256 == 0
    assert pkv.workspace_bytes(cfg, 65, 4096) == 0


def test_workload_generator_is_seeded_and_shaped():
    w = workloads.scaled(workloads.MISTRAL_RAGGED, num_layers=2, batch=3)
    lens = w.seq_lens()
    assert lens == w.seq_lens() and all(4096 <= n <= 16384 for n in lens)
    w2 = workloads.scaled(workloads.LLAMA2_7B, num_layers=2, seq_len=300)
    a = workloads.make_layer(w2, 1)
    b = workloads.make_layer(w2, 1)
    assert (a.k == b.k).all() and (a.q_win == b.q_win).all()
    assert a.k.shape == (1, 32, 300, 128) and a.q_win.shape == (1, 32, 32, 128)
    assert workloads.checksum(a.k) == workloads.checksum(b.k)
    assert len(a.planted[0]) == 4 + 16
