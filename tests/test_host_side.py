"""Host-side logic that needs no GPU: the C ABI's exports and argument checks, the multi-rank
bookkeeping (gloo, two processes), and the benchmark's CPU-oracle arm."""
import ctypes
import json
import os
import re
import socket
import subprocess
import sys

import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HAS_GPU = torch.cuda.is_available()


@pytest.fixture(scope="module")
def fef():
    import paper_2605_14305_b200 as lib

    lib.load(build_if_missing=True)
    return lib


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "fef.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(fef_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(fef):
    names = _declared_functions()
    assert "fef_spec_verify" in names and "fef_remask_select" in names and len(names) >= 9
    lib = fef.load()
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(fef.EXPORTS) == names


def test_status_strings(fef):
    seen = set()
    for code in range(0, 10):
        s = fef.fef_status_string(code)
        assert s and s != "unknown status"
        seen.add(s)
    assert len(seen) == 10
    assert fef.fef_status_string(1234) == "unknown status"


def test_header_constants_match_binding(fef):
    text = open(os.path.join(ROOT, "include", "fef.h")).read()
    assert int(re.search(r"#define FEF_MAX_K (\d+)", text).group(1)) == fef.FEF_MAX_K
    assert int(re.search(r"#define FEF_MAX_REMASK_L (\d+)", text).group(1)) == fef.FEF_MAX_REMASK_L
    assert re.search(r"#define FEF_STATIC_SCRATCH_BYTES \(8u << 20\)", text) and fef.FEF_STATIC_SCRATCH_BYTES == 8 << 20
    enum = dict(re.findall(r"(FEF_(?:OK|ERR_[A-Z_]+)) = (\d+)", text))
    for name, val in enum.items():
        assert getattr(fef, name) == int(val)


@pytest.mark.skipif(HAS_GPU, reason="uses placeholder addresses; only meaningful where no kernel can launch")
def test_argument_checks_return_before_touching_the_device(fef):
    """Every check below fails on the host, before any CUDA call; the placeholder addresses are
    never dereferenced.  With valid arguments and no device the answer is FEF_ERR_CUDA."""
    lib = fef.load()
    A = 0x1000  # 16-byte aligned placeholder
    def verify(q=A, p=A, tok=A, rl=None, B=2, K=4, V=64, ld=64, dt=0, T=1.0, al=A, tk=A, cf=A, ws=A, wsb=1 << 20):
        return lib.fef_spec_verify(q, p, tok, rl, B, K, V, ld, dt, T, 1, 1, al, tk, cf, ws, wsb, None, None)
    assert verify(dt=7) == fef.FEF_ERR_DTYPE
    assert verify(q=None) == fef.FEF_ERR_INVALID_ARG
    assert verify(cf=None) == fef.FEF_ERR_INVALID_ARG
    assert verify(B=0) == fef.FEF_ERR_INVALID_ARG
    assert verify(K=65) == fef.FEF_ERR_INVALID_ARG
    assert verify(V=0) == fef.FEF_ERR_INVALID_ARG
    assert verify(ld=63) == fef.FEF_ERR_INVALID_ARG
    assert verify(T=-0.5) == fef.FEF_ERR_INVALID_ARG
    assert verify(T=float("nan")) == fef.FEF_ERR_INVALID_ARG
    assert verify(q=A + 4) == fef.FEF_ERR_ALIGNMENT
    assert verify(V=10, ld=10) == fef.FEF_ERR_ALIGNMENT           # 40-byte fp32 rows
    assert verify(V=10, ld=12, dt=1) == fef.FEF_ERR_ALIGNMENT     # 24-byte bf16 rows
    assert verify() == fef.FEF_ERR_CUDA                           # nothing to run on
    assert lib.fef_remask_select(None, A, 1, 8, 2, A, A, None) == fef.FEF_ERR_INVALID_ARG
    assert lib.fef_remask_select(A, A, 1, 8193, 2, A, A, None) == fef.FEF_ERR_INVALID_ARG
    assert lib.fef_remask_select(A, A, 1, 8, -1, A, A, None) == fef.FEF_ERR_INVALID_ARG
    assert lib.fef_remask_select(A, A, 1, 8, 2, A, A, None) == fef.FEF_ERR_CUDA
    # the calls with a device-resident round counter need the counter
    assert lib.fef_spec_verify_at_round(A, A, A, None, None, 2, 4, 64, 64, 0, 1.0, 1, 1, None, A, A, A, A, 1 << 20, None,
                                        None) == fef.FEF_ERR_INVALID_ARG
    assert lib.fef_draft_sample_at_round(A, None, 2, 4, 64, 64, 0, 1.0, 1, 1, None, A, None, A, 1 << 20, None,
                                         None) == fef.FEF_ERR_INVALID_ARG
    assert lib.fef_loop_advance_round(None, None, 0, None) == fef.FEF_ERR_INVALID_ARG
    assert lib.fef_loop_advance_round(A, A, 0, None) == fef.FEF_ERR_INVALID_ARG
    # loop bookkeeping
    assert lib.fef_loop_next_window(None, 1, 8, 4, A, A, A, None) == fef.FEF_ERR_INVALID_ARG
    assert lib.fef_loop_next_window(A, 1, 0, 4, A, A, A, None) == fef.FEF_ERR_INVALID_ARG
    assert lib.fef_loop_next_window(A, 1, 8, 65, A, A, A, None) == fef.FEF_ERR_INVALID_ARG
    assert lib.fef_loop_commit(A, A, A, A, A, 1, 8, 4, A, A, None, A, None) == fef.FEF_ERR_INVALID_ARG
    assert lib.fef_loop_remask(None, A, 1, 8, 2, A, A, A, None) == fef.FEF_ERR_INVALID_ARG
    # vocabulary-parallel calls: sampling mode only, slice offsets in whole 16-byte vectors
    def stats(T=1.0, off=0, V=64, ld=64, st=A):
        return lib.fef_vp_local_stats(A, A, A, None, 2, 4, V, ld, 0, T, off, st, A, 1 << 20, None, None)
    assert stats(T=0.0) == fef.FEF_ERR_INVALID_ARG
    assert stats(off=4) == fef.FEF_ERR_INVALID_ARG
    assert stats(off=-8) == fef.FEF_ERR_INVALID_ARG
    assert stats(st=None) == fef.FEF_ERR_INVALID_ARG
    assert stats(V=10, ld=10) == fef.FEF_ERR_ALIGNMENT
    assert stats() == fef.FEF_ERR_CUDA
    assert lib.fef_vp_accept(A, 0, A, None, 2, 4, 64, 0, 1.0, 1, 1, A, A, A, A, None, None) == fef.FEF_ERR_INVALID_ARG
    assert lib.fef_vp_accept(A, 2, A, None, 2, 4, 0, 0, 1.0, 1, 1, A, A, A, A, None, None) == fef.FEF_ERR_INVALID_ARG
    assert lib.fef_vp_finish(A, 2, None, 2, 4, 0, 1.0, A, A, None) == fef.FEF_ERR_INVALID_ARG
    assert lib.fef_vp_local_residual(A, A, A, 2, 4, 64, 64, 0, 1.0, 1, 1, 12, A, A, 1 << 20, None) == fef.FEF_ERR_INVALID_ARG
    assert lib.fef_vp_task_bytes(0) == 0 and lib.fef_vp_task_bytes(3) == 96
    assert fef.fef_spec_verify_workspace_bytes(64, 32, 126464, torch.bfloat16) == 0  # no device: no size
    with pytest.raises(RuntimeError):
        fef.fef_spec_verify(torch.zeros(1, 1, 8), torch.zeros(1, 1, 8), torch.zeros(1, 1, dtype=torch.int32), 1.0, 0, 0)


def test_shard_and_rate_helpers():
    from paper_2605_14305_b200 import dist_util as du

    for total in (0, 1, 7, 64, 65):
        for world in (1, 2, 3, 8):
            spans = [du.shard_windows(total, r, world) for r in range(world)]
            assert spans[0][0] == 0 and sum(c for _, c in spans) == total
            for (f0, c0), (f1, _) in zip(spans, spans[1:]):
                assert f0 + c0 == f1
            assert max(c for _, c in spans) - min(c for _, c in spans) <= 1
    assert len({du.rank_seed(5, r) for r in range(8)}) == 8 and du.rank_seed(5, 0) == 5
    assert du.aggregate_rate(2048, 10, 2.0, 4) == 2048 * 4 * 10 / 2e-3
    assert du.max_over_ranks([1.0, 2.0]) == [1.0, 2.0]


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


_GLOO_WORKER = r"""
import os, sys, json
sys.path.insert(0, %r)
import numpy as np, torch, torch.distributed as dist
from paper_2605_14305_b200 import dist_util as du, synth
import oracle

dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
# each rank times "its" work; the job time is the slowest rank's
got = du.max_over_ranks([10.0 + rank, 5.0 - rank])
assert got == [10.0 + world - 1, 5.0], got
# the windows of one logical batch, sharded: every rank verifies its share with the oracle,
# drawing random numbers as global window batch_offset + b; gathered, it equals the unsharded run
w = synth.TINY.with_(B=6, K=3, V=40, noise_std=1.0)
q, p, tok = synth.make_call(w, seed=9)
first, count = du.shard_windows(w.B, rank, world)
part = oracle.spec_verify(q[first:first + count], p[first:first + count], tok[first:first + count], 1.0, 7, 3,
                          batch_offset=first)
mine = torch.full((w.B, w.K), -7, dtype=torch.int32)
mine[first:first + count] = torch.as_tensor(part["tokens"])
dist.all_reduce(mine, op=dist.ReduceOp.MAX)
whole = oracle.spec_verify(q, p, tok, 1.0, 7, 3)
assert (mine.numpy() == whole["tokens"]).all()
# replicas: distinct seeds per rank give different draws on identical inputs
a = oracle.spec_verify(q, p, tok, 1.0, du.rank_seed(7, rank), 3)["tokens"]
gathered = [torch.zeros((w.B, w.K), dtype=torch.int32) for _ in range(world)]
dist.all_gather(gathered, torch.as_tensor(a))
assert any((gathered[0] != g).any() for g in gathered[1:])
# vocabulary-parallel exchange: every rank reduces its slice to (reference, sum) per row; gathered
# rank-major (the layout fef_vp_accept reads) and folded, they give the full rows' normalisers
from paper_2605_14305_b200.vocab_parallel import shard_vocab, STATS_PER_ROW
rows = q.reshape(-1, w.V).double()
off, width = shard_vocab(w.V, world)[rank]
sl = rows[:, off:off + width]
mine = torch.zeros((rows.shape[0], STATS_PER_ROW), dtype=torch.float64)
mine[:, 0] = sl.max(dim=1).values
mine[:, 1] = torch.exp2(sl - mine[:, :1]).sum(dim=1)
everyone = torch.empty((world * mine.shape[0], STATS_PER_ROW), dtype=torch.float64)
dist.all_gather_into_tensor(everyone, mine)
everyone = everyone.reshape(world, mine.shape[0], STATS_PER_ROW)
M = everyone[:, :, 0].max(dim=0).values
S = (everyone[:, :, 1] * torch.exp2(everyone[:, :, 0] - M)).sum(dim=0)
assert torch.allclose(M + torch.log2(S), torch.log2(torch.exp2(rows).sum(dim=1)), rtol=1e-12, atol=1e-12)
assert off %% 8 == 0 and sum(wd for _, wd in shard_vocab(w.V, world)) == w.V
rate = du.aggregate_rate(w.B * w.K, 4, got[0], world)
if rank == 0:
    print(json.dumps({"ok": True, "rate": rate}))
dist.destroy_process_group()
"""


def test_two_rank_gloo_bookkeeping(tmp_path):
    script = tmp_path / "gloo_worker.py"
    script.write_text(_GLOO_WORKER % ROOT)
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
           "--master-addr", "127.0.0.1", "--master-port", str(_free_port()), str(script)]
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=240, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    line = [l for l in r.stdout.splitlines() if l.startswith("{")][-1]
    out = json.loads(line)
    assert out["ok"] and abs(out["rate"] - 18 * 2 * 4 / (11.0e-3)) < 1e-6


def test_bench_reference_arm_single_and_two_ranks():
    """`bench.py --impl reference` times the CPU oracle; under torchrun only rank 0 prints."""
    base = [os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny", "--steps", "3", "--warmup", "1"]
    r = subprocess.run([sys.executable] + base, capture_output=True, text=True, timeout=240, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    d = json.loads(r.stdout.strip().splitlines()[-1])
    assert d["impl"] == "reference" and d["value"] > 0 and d["unit"] == "positions/s" and d["steps"] == 3
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] == 1
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["e2e"]["value"] == d["value"]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2", "--master-addr",
           "127.0.0.1", "--master-port", str(_free_port())] + base + ["--gpus", "2"]
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=240, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1 and json.loads(lines[0])["impl"] == "reference"


def test_decode_loop_driver_with_the_oracle_as_backend():
    """Algorithm 2's outer loop (windows over unresolved positions, commit, LowConf re-masking) run on
    the CPU with the oracle behind both calls: everything ends resolved and step budgets hold."""
    import numpy as np

    import oracle
    from paper_2605_14305_b200 import synth
    from paper_2605_14305_b200.decode_loop import run_decode_loop

    w = synth.TINY.with_(B=3, K=4, V=50, noise_std=1.0)
    L, n_steps, k = 10, 3, 2

    def logits_fn(rnd, window, row_len):
        return synth.make_logits(w, seed=100 + rnd)

    def draft_fn(q, rnd):
        return synth.sample_draft_tokens(q, 1.0, 200 + rnd)

    calls = []

    def verify_fn(q, p, tok, rl, rnd):
        r = oracle.spec_verify(q, p, tok, 1.0, 1, rnd, row_len=rl)
        calls.append(rl.numpy().copy())
        return r["accept_len"], r["tokens"], r["conf"]

    def select_fn(conf, mask, kk):
        return oracle.remask_select(conf, mask, kk)

    out = run_decode_loop(w.B, L, w.K, n_steps, k, logits_fn, draft_fn, verify_fn, select_fn, device="cpu")
    assert (out["tokens"] >= 0).all() and (out["conf"] >= 0).all()
    assert out["rounds"] == len(calls) and sum(out["committed_per_round"]) == w.B * (L + (n_steps - 1) * k)
    assert all((c <= w.K).all() for c in calls)
    # after the first denoising step only the k re-masked positions per row are unresolved
    first_redo = next(i for i, c in enumerate(calls) if i > 0 and (c == k).all() and (calls[i - 1] != k).any())
    assert first_redo >= L // w.K


_VP_WORKER = r"""
import ctypes, json, sys
sys.path.insert(0, %r)
import torch, torch.distributed as dist
from paper_2605_14305_b200 import vocab_parallel as vp

dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
B, K, Vloc = 3, 4, 16


class FakeLibrary:
    # Stand-in for the loaded library: records the order of the calls, fills this rank's outputs with
    # values that name the rank, and checks what the gathers hand to the next step.
    def __init__(self):
        self.calls = []

    def fef_spec_verify_workspace_bytes(self, B_, K_, V_, code):
        return 4096

    def fef_vp_task_bytes(self, B_):
        return 32 * B_

    def _view(self, ptr, n, ctype):
        return (ctype * n).from_address(ptr)

    def fef_vp_local_stats(self, q, p, tok, row_len, B_, K_, V_, ld, code, T, offset, stats, ws, wsb, status, stream):
        self.calls.append("stats")
        assert (B_, K_, V_, ld) == (B, K, Vloc, Vloc) and offset == rank * Vloc and wsb >= 4096 and stream == 0
        s = self._view(stats, B * K * vp.STATS_PER_ROW, ctypes.c_double)
        for i in range(len(s)):
            s[i] = 1000.0 * rank + i
        return 0

    def fef_vp_accept(self, stats_all, ranks, tok, row_len, B_, K_, V_total, code, T, seed, step, accept_len, tokens, conf,
                      tasks, status, stream):
        self.calls.append("accept")
        assert ranks == world and V_total == world * Vloc and (seed, step) == (77, 5)
        n = B * K * vp.STATS_PER_ROW
        s = self._view(stats_all, world * n, ctypes.c_double)
        for r in range(world):          # rank-major: rank r's block follows rank r - 1's
            assert s[r * n] == 1000.0 * r and s[r * n + n - 1] == 1000.0 * r + n - 1
        a = self._view(accept_len, B, ctypes.c_int32)
        for b in range(B):
            a[b] = b
        return 0

    def fef_vp_local_residual(self, q, p, tasks, B_, K_, V_, ld, code, T, seed, step, offset, cand, ws, wsb, stream):
        self.calls.append("residual")
        assert offset == rank * Vloc and (seed, step) == (77, 5)
        c = self._view(cand, B * vp.CANDIDATE_BYTES, ctypes.c_uint8)
        for i in range(len(c)):
            c[i] = (17 * rank + i) %% 251
        return 0

    def fef_vp_finish(self, cand_all, ranks, tasks, B_, K_, code, T, tokens, conf, stream):
        self.calls.append("finish")
        assert ranks == world
        n = B * vp.CANDIDATE_BYTES
        c = self._view(cand_all, world * n, ctypes.c_uint8)
        for r in range(world):
            assert c[r * n] == (17 * r) %% 251 and c[r * n + n - 1] == (17 * r + n - 1) %% 251
        return 0


lib = FakeLibrary()
q = torch.zeros((B, K, Vloc))
tok = torch.zeros((B, K), dtype=torch.int32)
out = vp.fef_spec_verify_vocab_parallel(q, q.clone(), tok, 1.0, 77, 5, rank * Vloc, world * Vloc, lib=lib)
assert lib.calls == ["stats", "accept", "residual", "finish"], lib.calls
assert out.accept_len.tolist() == [0, 1, 2]
if rank == 0:
    print(json.dumps({"ok": True}))
"""


def test_vocab_parallel_orchestration_over_gloo_with_a_stand_in_library(tmp_path):
    """The four steps of the vocabulary-parallel call and its two all-gathers, driven on two CPU
    ranks (gloo) with a stand-in for the library: call order, arguments, and the rank-major layout
    of what each gather hands to the following step."""
    script = tmp_path / "vp_worker.py"
    script.write_text(_VP_WORKER % ROOT)
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
           "--master-addr", "127.0.0.1", "--master-port", str(_free_port()), str(script)]
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=240, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-3000:]
    assert json.loads([l for l in r.stdout.splitlines() if l.startswith("{")][-1])["ok"]


def test_bench_gpus_flag_starts_ranks_itself(tmp_path):
    """`bench.py --gpus 2` run by hand (no WORLD_SIZE) re-launches itself as two ranks; rank 0 alone prints."""
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny", "--steps", "2",
           "--warmup", "1", "--gpus", "2"]
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=240, cwd=ROOT, env=env)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and "parallelism" in d and "parallelism" not in d["config"]
