"""A producer of the hidden states that signals "dependents may start" before its last store.

Library kernels of that kind exist (GEMMs and fused normalisations built for programmatic dependent
launch), and a caller cannot see it from outside.  By default a kvzap call must therefore read its
inputs only after everything ahead of it in the stream has completed, although its kernels are
launched with the attribute that lets them start early.  The test puts such a producer (a small
kernel compiled here from tests/helpers/early_producer.cu: signal, idle for ~0.2 ms, then write the
hidden states) directly ahead of a scoring call, a fused prefill call and a decode step, and checks
that the results are those of the NEW hidden states, bit for bit.
"""
import ctypes
import os
import shutil
import subprocess

import pytest
import torch

from paper_2601_07891_b200 import synth

pytestmark = pytest.mark.gpu

HERE = os.path.dirname(os.path.abspath(__file__))


@pytest.fixture(scope="module")
def producer():
    nvcc = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(nvcc):
        pytest.skip("nvcc is needed to build the test's producer kernel")
    out_dir = os.path.join(HERE, "_build")
    os.makedirs(out_dir, exist_ok=True)
    lib = os.path.join(out_dir, "libearly_producer.so")
    subprocess.run([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O2", "-shared", "-Xcompiler", "-fPIC",
                    "-o", lib, os.path.join(HERE, "helpers", "early_producer.cu")], check=True)
    L = ctypes.CDLL(lib)
    L.launch_early_producer.restype = ctypes.c_int
    L.launch_early_producer.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_longlong, ctypes.c_longlong,
                                        ctypes.c_void_p]

    def launch(src, dst, delay_cycles=400000):
        assert src.numel() * src.element_size() % 16 == 0
        rc = L.launch_early_producer(src.data_ptr(), dst.data_ptr(), src.numel() * src.element_size(), delay_cycles,
                                     torch.cuda.current_stream().cuda_stream)
        assert rc == 0
    return launch


@pytest.fixture(scope="module")
def binding():
    from paper_2601_07891_b200 import binding as b
    b.load()
    return b


@pytest.mark.parametrize("d_model,hidden,T", [(1024, 256, 300), (1024, 256, 40000), (1024, 0, 2000), (512, 0, 30000)])
def test_scoring_and_fused_prefill_read_hidden_after_an_early_signalling_producer(binding, producer, d_model, hidden, T):
    H, D, tau, w = 8, 64, 0.2, 32
    ctx = binding.Kvzap(d_model, hidden, H, D, 1, T)          # default flags: producers are not trusted
    wts = synth.mlp_weights(d_model, hidden, H, 5, "cuda", 0.3) if hidden else synth.linear_weights(d_model, H, 5, "cuda", 0.3)
    ctx.set_weights(0, *wts)
    X_old = synth.hidden_states(T, d_model, 1, "cuda")
    X_new = synth.hidden_states(T, d_model, 2, "cuda")
    K, V = synth.keys_values(H, T, D, 3, "cuda")
    want = ctx.score(0, X_new)
    Ko_ref, Vo_ref, len_ref = ctx.prefill_fused(0, X_new, K, V, tau, w)
    torch.cuda.synchronize()
    for call in ("score", "fused"):
        for rep in range(3):
            hidden_buf = X_old.clone()
            torch.cuda.synchronize()
            producer(X_new, hidden_buf)
            if call == "score":
                got = ctx.score(0, hidden_buf)
                torch.cuda.synchronize()
                assert torch.equal(got.view(torch.int32), want.view(torch.int32)), (call, rep)
            else:
                Ko, Vo, ln = ctx.prefill_fused(0, hidden_buf, K, V, tau, w)
                torch.cuda.synchronize()
                assert torch.equal(ln, len_ref), (call, rep)
                for h in range(H):
                    n = int(ln[0, h])
                    assert torch.equal(Ko[h, :n].view(torch.int16), Ko_ref[h, :n].view(torch.int16))
                    assert torch.equal(Vo[h, :n].view(torch.int16), Vo_ref[h, :n].view(torch.int16))
    assert ctx.poll_status() == 0
    ctx.close()


def test_decode_step_reads_hidden_after_an_early_signalling_producer(binding, producer):
    d_model, hidden, H, D, w, P, B, L, tau = 512, 256, 8, 64, 8, 4, 5, 3, 0.1
    ctx = binding.Kvzap(d_model, hidden, H, D, L, max_tokens=128)
    for l in range(L):
        ctx.set_weights(l, *synth.mlp_weights(d_model, hidden, H, 20 + l, "cuda", 0.3))
    n_pool = B * L * H * 8
    K_pool = torch.zeros(n_pool, P, D, dtype=torch.bfloat16, device="cuda")
    V_pool = torch.zeros_like(K_pool)
    cache = binding.kvzap_cache_create(ctx.handle, B, w, P, K_pool, V_pool, 8)
    X_old = synth.hidden_states(L * B, d_model, 1, "cuda").view(L, B, d_model)
    for step in range(6):
        X_new = synth.hidden_states(L * B, d_model, 10 + step, "cuda").view(L, B, d_model)
        Kn, Vn = synth.keys_values(L * B, H, D, 30 + step, "cuda")
        want = torch.stack([ctx.score(l, X_new[l]) for l in range(L)])
        buf = X_old.clone()
        sc = torch.empty(L, B, H, dtype=torch.float32, device="cuda")
        torch.cuda.synchronize()
        producer(X_new, buf)
        binding.kvzap_decode_step(ctx.handle, cache, 0, L, buf, Kn.view(L, B, H, D), Vn.view(L, B, H, D), tau, sc)
        torch.cuda.synchronize()
        assert torch.allclose(sc, want, atol=1e-5, rtol=0), step          # another kernel layout: not the same bits
    assert ctx.poll_status() == 0
    binding.kvzap_cache_destroy(cache)
    ctx.close()
