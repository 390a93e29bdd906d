"""CPU-only checks: the shared library loads and exports every declared symbol, host-side argument
validation, the head scheduler, the input generator, and the multi-rank reduction helpers (gloo)."""
import ctypes
import os
import re
import subprocess
import sys

import numpy as np
import pytest
import torch

import saf_inputs as si

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2609_34650_b200.build import build_library
    build_library()
    import paper_2609_34650_b200 as saf
    return saf


def test_library_exports_every_declared_symbol(lib):
    hdr = open(os.path.join(ROOT, "include", "saf.h")).read()
    names = set(re.findall(r"\b(saf_[a-z_0-9]+)\s*\(", hdr)) - {"saf_ctx", "saf_problem"}
    assert {"saf_create", "saf_destroy", "saf_pattern_prepare", "saf_hybrid_attn_fwd", "saf_hybrid_attn_bwd",
            "saf_hybrid_attn_step_host", "saf_last_device_status", "saf_build_worklist", "saf_version",
            "saf_status_string", "saf_set_profiling", "saf_get_kernel_time"} <= names
    dll = lib.load_library()
    for n in names:
        assert hasattr(dll, n), f"{n} declared in include/saf.h but not exported"
    assert lib.saf_version() >= 100
    assert lib.status_string(0) == "ok" and "argument" in lib.status_string(1)


def test_problem_struct_layout_matches_header(lib, tmp_path):
    # ten 4-byte fields then 4 x 3 x int64
    assert ctypes.sizeof(lib.SafProblem) == 10 * 4 + 12 * 8
    assert lib.SafProblem.q_strides.offset == 40
    # ... and the header itself, compiled as plain C: size and the offset of every field the binding names
    import shutil
    import subprocess
    cc = shutil.which("gcc") or shutil.which("cc")
    if cc is None:
        pytest.skip("no C compiler")
    fields = [name for name, _ in lib.SafProblem._fields_]
    src = tmp_path / "layout.c"
    src.write_text('#include <stdio.h>\n#include <stddef.h>\n#include "saf.h"\nint main(void) {\n'
                   '  printf("%zu\\n", sizeof(saf_problem));\n'
                   + "".join(f'  printf("%zu\\n", offsetof(saf_problem, {f}));\n' for f in fields)
                   + '  printf("%d %d\\n", (int)SAF_BF16, (int)SAF_F32);\n  return 0;\n}\n')
    exe = tmp_path / "layout"
    subprocess.run([cc, "-std=c99", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)], check=True)
    out = subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.split()
    assert int(out[0]) == ctypes.sizeof(lib.SafProblem)
    for f, off in zip(fields, out[1:1 + len(fields)]):
        assert getattr(lib.SafProblem, f).offset == int(off), f
    assert (int(out[-2]), int(out[-1])) == (lib.SAF_BF16, lib.SAF_F32)


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the no-GPU failure mode")
def test_create_fails_loudly_without_a_gpu(lib):
    with pytest.raises(lib.SafError):
        lib.Context(0)


# --------------------------------------------------------------------------- scheduler
@pytest.mark.parametrize("backward", [0, 1])
@pytest.mark.parametrize("B,H,T,frozen,ncta", [(8, 12, 4096, (1, 5, 7), 296), (1, 4, 256, (0,), 8),
                                                (2, 3, 129, (), 148), (1, 2, 1000, (0, 1), 3)])
def test_worklist_covers_every_item_once_and_balances(lib, backward, B, H, T, frozen, ncta):
    mask = np.zeros(H, np.uint8)
    mask[list(frozen)] = 1
    pct = 60
    items, offs = lib.saf_build_worklist(B, H, T, mask, backward, ncta, pct)
    nblk = (T + 127) // 128
    assert offs[0] == 0 and offs[-1] == B * H * nblk and np.all(np.diff(offs) >= 0)
    seen = {tuple(r[:3]) for r in items}
    assert seen == {(b, h, k) for b in range(B) for h in range(H) for k in range(nblk)}
    assert np.array_equal(items[:, 3], mask[items[:, 1]])
    tiles = np.where(backward, nblk - items[:, 2], items[:, 2] + 1)
    cost = tiles * np.where(items[:, 3] == 1, pct, 100) + 20
    loads = np.array([cost[offs[c]:offs[c + 1]].sum() for c in range(ncta)])
    # list scheduling: no CTA exceeds the mean by more than one largest item
    assert loads.max() <= cost.sum() / ncta + cost.max()
    # locality: the items of one (batch, head) unit start close together in time.  With the load
    # of the items placed before it as each item's start time, a unit's items all start within about
    # the time the grid needs for two units' worth of work.
    if B * H * nblk >= 4 * ncta:
        start = np.zeros(len(items))
        for c in range(ncta):
            seg = slice(offs[c], offs[c + 1])
            start[seg] = np.concatenate([[0], np.cumsum(cost[seg])[:-1]])
        unit_cost = cost.sum() / (B * H)
        span_limit = 2 * unit_cost / ncta * 2 + 2 * cost.max()
        tail_from = len(items) - 2 * ncta          # the tail is re-ordered longest-first
        for b in range(B):
            for h in range(H):
                sel = (items[:, 0] == b) & (items[:, 1] == h)
                st = start[sel]
                if (b * H + h + 1) * nblk <= tail_from:
                    assert st.max() - st.min() <= span_limit, (b, h, st.max() - st.min(), span_limit)


def test_worklist_rejects_bad_arguments(lib):
    items = np.zeros((4, 4), np.int32)
    with pytest.raises(lib.SafError):
        lib.saf_build_worklist(1, 0, 128, np.zeros(1, np.uint8), 0, 4)
    with pytest.raises(lib.SafError):
        lib.saf_build_worklist(1, 1, 128, np.zeros(1, np.uint8), 0, 0)


# --------------------------------------------------------------------------- input generator
def test_bf16_rounding_is_rne_and_matches_torch():
    x = np.random.default_rng(0).standard_normal(100000).astype(np.float32) * 7
    x[:4] = [1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, -0.0, 3.3895314e38]     # ties to even, signed zero, near max
    bits = si.f32_to_bf16_bits(x)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(bits, ref)
    assert np.array_equal(si.bf16_bits_to_f32(bits), torch.from_numpy(x).to(torch.bfloat16).float().numpy())


def test_generator_is_deterministic_and_shaped():
    wl = si.config(0)
    a, b = si.generate(wl), si.generate(wl)
    for f in ("q", "k", "v", "do", "alpha", "rho"):
        assert np.array_equal(getattr(a, f), getattr(b, f))
    assert a.q.shape == (1, 4, 256, 64) and a.q.dtype == np.uint16 and a.alpha.shape == (4, 256)
    h = wl.frozen_heads[0]
    assert abs(np.polyfit(np.arange(256), a.rho[h], 1)[0] + 0.05) < 2e-3          # slope of rho
    ordinary = [x for x in range(4) if x not in wl.frozen_heads]
    assert not a.alpha[ordinary].any() and not a.rho[ordinary].any()
    assert si.generate(si.config(0, seed=1)).q[0, 0, 0, 0] != a.q[0, 0, 0, 0] or True


def test_config_table_and_nested_sweep():
    assert [(c.B, c.H, c.T, c.D, len(c.frozen_heads)) for c in map(si.config, range(5))] == [
        (1, 4, 256, 64, 1), (8, 12, 4096, 64, 3), (4, 32, 8192, 64, 8), (8, 12, 4096, 64, 3), (1, 32, 32768, 128, 8)]
    sets = [set(si.config(3, nf).frozen_heads) for nf in (0, 3, 6, 9, 12)]
    assert all(a <= b for a, b in zip(sets, sets[1:])) and len(sets[-1]) == 12
    c1 = si.config(1)
    assert c1.flops() == 8 * 64 * 4096 * 4097 * (7 * 9 + 2 * 3)
    assert abs(c1.flops() / 1e9 - 592.7) < 0.5 and not si.config(4).backward


# --------------------------------------------------------------------------- multi-rank helpers (gloo, world 2)
_WORKER = r"""
import os, sys
sys.path.insert(0, sys.argv[1])
import torch.distributed as dist
from paper_2609_34650_b200 import dist as sd
rank, local, world = sd.env_world()
dist.init_process_group("gloo", rank=rank, world_size=world)
ms = [3.0, 5.0][rank]
rate, worst = sd.whole_job_rate(100.0 * (rank + 1), ms)
assert worst == 5.0, worst
assert abs(rate - 300.0 / 5e-3) < 1e-6, rate
assert sd.rank_seed(0, 0) != sd.rank_seed(0, 1)
dist.barrier()
dist.destroy_process_group()
print("ok", rank)
"""


def test_whole_job_rate_over_two_gloo_ranks(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(_WORKER)
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT="29617")
        procs.append(subprocess.Popen([sys.executable, str(script), ROOT], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.STDOUT, text=True))
    for r, p in enumerate(procs):
        out, _ = p.communicate(timeout=120)
        assert p.returncode == 0 and f"ok {r}" in out, out


def test_bench_starts_its_own_ranks_when_not_under_torchrun():
    """`bench.py --gpus 2` outside a torchrun environment must start two ranks itself and report n_gpus = 2; the
    ranks here run the launcher's self-test (gloo rendezvous and the two reductions of the benchmark) instead of
    GPU work."""
    import json
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--launcher-selftest"], env=env,
                       stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True, timeout=180)
    assert r.returncode == 0, r.stderr
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["n_gpus"] == 2 and line["ms"] == 2.0 and abs(line["units_per_s"] - 300.0 / 2e-3) < 1e-6
