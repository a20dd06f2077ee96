"""Memory-safety evidence on the GPU without a memory checker: every buffer a layer call writes (packed
blobs, workspace, routing outputs, output rows) sits between guard zones filled with a pattern, and the
guards must be intact after full-size calls of both expert kernels; and a call repeated on a workspace
overwritten with garbage must give the same bits (no read of stale scratch, no order dependence on the
work queue)."""
import pytest
import torch

from paper_2504_15299_b200 import synth

pytestmark = pytest.mark.gpu

GUARD = 4096          # bytes on either side (keeps the 256-byte / 16-byte alignments of the inner buffer)
PATTERN = 0xA5


@pytest.fixture(scope="module")
def B():
    from paper_2504_15299_b200 import binding, build
    build.build_library()
    binding.lib()
    return binding


class Guarded:
    """A device byte buffer with guard zones; `.inner` is the part handed to the library."""

    def __init__(self, nbytes: int):
        self.n = nbytes
        self.raw = torch.full((nbytes + 2 * GUARD,), PATTERN, dtype=torch.uint8, device="cuda")
        assert self.raw.data_ptr() % 256 == 0
        self.inner = self.raw[GUARD:GUARD + nbytes]

    def view(self, dtype, shape):
        return self.inner.view(dtype).reshape(shape)

    def intact(self) -> bool:
        lo, hi = self.raw[:GUARD], self.raw[GUARD + self.n:]
        return bool((lo == PATTERN).all().item()) and bool((hi == PATTERN).all().item())


def guarded_layer(B, cfg, wl):
    blobs, guards = [], []
    for e in range(wl.n_experts + wl.n_shared):
        for m in range(3):
            rows, cols = synth.expert_matrix_shape(wl, m)
            g = Guarded(B.packed_bytes(cfg, rows, cols)[0])
            W = synth.expert_matrix(wl, e, m, device="cuda")
            B.pack_mwq(cfg, W, out=g.inner)
            del W
            blobs.append(g.inner)
            guards.append(g)
    torch.cuda.synchronize()
    return blobs, guards


@pytest.mark.parametrize("name,T", [("mixtral_decode", 64), ("mixtral_decode", 1), ("mixtral_prefill", 2048),
                                    ("finegrained", 256)])
def test_guard_zones_survive_and_reruns_are_bit_identical(B, name, T):
    wl = synth.WORKLOADS[name]
    cfg = B.Config.from_workload(wl)
    blobs, guards = guarded_layer(B, cfg, wl)
    assert all(g.intact() for g in guards)                      # packing stayed inside its blobs
    x = synth.tokens_bf16(wl, T, "cuda")
    fb = synth.forced_bit_idx(wl, T, "cuda")
    kw = {"forced_bit_idx": fb}
    if wl.zipf_logits:
        kw["logits"] = synth.zipf_logits(wl, T, "cuda")
    else:
        kw["gate_w"] = synth.gate_weight_bf16(wl, "cuda")
    A, K = T * wl.top_k, len(wl.bits)
    ws = Guarded(B.workspace_bytes(cfg, T))
    yg = Guarded(T * wl.d_model * 2)
    y = yg.view(torch.bfloat16, (T, wl.d_model))
    # routing outputs in guarded buffers too, then the layer from that routing
    r_bufs = [Guarded(A * 4), Guarded(A * 4), Guarded(A), Guarded(A * 4), Guarded(A * 4), Guarded((wl.n_experts * K + 1) * 4)]
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    pre = B.RouteResult(r_bufs[0].view(torch.int32, (T, wl.top_k)), r_bufs[1].view(torch.float32, (T, wl.top_k)),
                        r_bufs[2].view(torch.int8, (T, wl.top_k)), r_bufs[3].view(torch.int32, (A,)),
                        r_bufs[4].view(torch.int32, (A,)), r_bufs[5].view(torch.int32, (wl.n_experts * K + 1,)), st)
    import ctypes
    B._check(B.lib().d2moe_route(ctypes.byref(cfg.c()), T, x.data_ptr(), B._ptr(kw.get("gate_w")), B._ptr(kw.get("logits")),
                                 None, fb.data_ptr(), pre.topk_idx.data_ptr(), pre.topk_w.data_ptr(), pre.bit_idx.data_ptr(),
                                 pre.perm.data_ptr(), pre.inv_perm.data_ptr(), pre.group_off.data_ptr(), st.data_ptr(),
                                 ws.inner.data_ptr(), ws.n, None), "d2moe_route")
    B.moe_forward(cfg, x, blobs, pre=pre, y=y, workspace=ws.inner, device_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    y_pre = y.clone()
    # the whole call (routing inside), twice, the workspace overwritten with garbage in between
    B.moe_forward(cfg, x, blobs, y=y, workspace=ws.inner, device_status=st, **kw)
    torch.cuda.synchronize()
    y1 = y.clone()
    ws.inner.fill_(0xFF)
    y.fill_(float("nan"))
    B.moe_forward(cfg, x, blobs, y=y, workspace=ws.inner, device_status=st, **kw)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    assert torch.equal(y1.view(torch.int16), y.view(torch.int16))             # bit-identical rerun
    assert torch.equal(y_pre.view(torch.int16), y.view(torch.int16))          # and identical with routing supplied
    assert bool(torch.isfinite(y.float()).all().item())
    for g in guards + r_bufs + [ws, yg]:
        assert g.intact()


_CHAIN_SCRIPT = r"""
import hashlib, sys, torch
from paper_2504_15299_b200 import binding as B, synth
out = []
for name, T in (("tiny", 24), ("mixtral_decode", 8)):
    wl = synth.WORKLOADS[name]
    cfg = B.Config.from_workload(wl)
    blobs = []
    for e in range(wl.n_experts + wl.n_shared):
        for m in range(3):
            blobs.append(B.pack_mwq(cfg, synth.expert_matrix(wl, e, m, device="cuda")))
    x = synth.tokens_bf16(wl, T, "cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    y = B.moe_forward(cfg, x, blobs, gate_w=synth.gate_weight_bf16(wl, "cuda"),
                      forced_bit_idx=synth.forced_bit_idx(wl, T, "cuda"), device_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    out.append(hashlib.sha256(y.view(torch.int16).cpu().numpy().tobytes()).hexdigest())
print("HASH", " ".join(out))
"""


def test_ordinary_launches_give_the_same_bits_as_the_dependent_launch_chain(B):
    """The kernels of a call are programmatic dependent launches; D2MOE_NO_PDL=1 (read once per process, hence the
    child processes) makes them ordinary launches.  Both must give the same output bits."""
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    hashes = []
    for flag in ("0", "1"):
        env = dict(os.environ, D2MOE_NO_PDL=flag, PYTHONPATH=root + os.pathsep + os.environ.get("PYTHONPATH", ""))
        r = subprocess.run([sys.executable, "-c", _CHAIN_SCRIPT], env=env, cwd=root, capture_output=True, text=True, timeout=600)
        assert r.returncode == 0, r.stderr[-2000:]
        line = [ln for ln in r.stdout.splitlines() if ln.startswith("HASH")]
        assert line, r.stdout[-2000:]
        hashes.append(line[-1])
    assert hashes[0] == hashes[1]
