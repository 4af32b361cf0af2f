"""Several verifiers at once: one context per host thread, each on its own CUDA stream, launching the library's
persistent kernels side by side on one GPU.  No kernel of the library waits for a kernel of another launch (a worker
only ever waits for work that a worker resident before it will hand on), so launches that overlap, or that have to
take turns on the SMs because of their shared memory, must all finish and give the oracle's digests and roots."""
import threading

import numpy as np
import pytest
import torch

import oracle
from paper_2510_23938_b200 import binding, inputs

pytestmark = pytest.mark.gpu

MIB = 1 << 20


def _host(t: torch.Tensor) -> np.ndarray:
    return t.cpu().numpy()


def test_three_contexts_on_three_streams_from_three_threads():
    if not torch.cuda.is_available():
        pytest.fail("the gpu-marked tests need a CUDA device")
    # (entry point, bytes, chunk): few chains (two-warp kernel), many chains (migrating kernel), SHA-384 pairs,
    # a ragged last chunk on the forked stream, and the one-chain-per-lane kernels
    jobs = [
        [("sha256", 768 * MIB, 4 * MIB), ("sha256", 64 * MIB + 4097, 64 << 10), ("rfc6962", 256 * MIB, 1 * MIB)],
        [("sha256", 1024 * MIB, 64 << 10), ("sha384", 300 * MIB + 77, 256 << 10), ("sha256", 512 * MIB, 4096)],
        [("sha384", 1024 * MIB, 256 << 10), ("sha512", 96 * MIB, 4096), ("sha256", 640 * MIB, 1 * MIB)],
    ]
    datas, wants = [], []
    threads = oracle.host_threads()
    for k, seq in enumerate(jobs):
        nmax = max(n for _, n, _ in seq)
        d = inputs.uniform_bytes(nmax, seed=9100 + k, device="cuda")
        h = _host(d)
        w = []
        for kind, n, chunk in seq:
            if kind == "sha256":
                dg = oracle.hash_chunks(h[:n], chunk, nthreads=threads); root = oracle.merkle_root(dg)
            elif kind == "rfc6962":
                dg = oracle.hash_chunks_rfc6962(h[:n], chunk, nthreads=threads); root = oracle.merkle_root_rfc6962(dg)
            elif kind == "sha384":
                dg = oracle.hash_chunks_sha384(h[:n], chunk, nthreads=threads); root = oracle.merkle_root_sha384(dg)
            else:
                dg = oracle.hash_chunks_sha512(h[:n], chunk, nthreads=threads); root = oracle.merkle_root_sha512(dg)
            w.append((dg, root))
        datas.append(d)
        wants.append(w)
    torch.cuda.synchronize()

    errors, start = [], threading.Barrier(len(jobs))

    def worker(k):
        try:
            torch.cuda.set_device(0)
            ctx = binding.Context(0)
            stream = torch.cuda.Stream()
            start.wait()
            for rep in range(3):
                outs = []
                for kind, n, chunk in jobs[k]:
                    d = datas[k][:n]
                    if kind == "sha256":
                        dg = ctx.hash_chunks(d, chunk, stream=stream); root = ctx.merkle_root(dg, stream=stream)
                    elif kind == "rfc6962":
                        dg = ctx.hash_chunks_rfc6962(d, chunk, stream=stream); root = ctx.merkle_root_rfc6962(dg, stream=stream)
                    elif kind == "sha384":
                        dg = ctx.hash_chunks_sha384(d, chunk, stream=stream); root = ctx.merkle_root_sha384(dg, stream=stream)
                    else:
                        dg = ctx.hash_chunks_sha512(d, chunk, stream=stream); root = ctx.merkle_root_sha512(dg, stream=stream)
                    outs.append((dg, root))          # no synchronisation between the calls of a thread
                stream.synchronize()
                for (dg, root), (wdg, wroot), job in zip(outs, wants[k], jobs[k]):
                    if not np.array_equal(_host(dg), wdg):
                        errors.append(f"thread {k} rep {rep} {job}: digests differ from the oracle")
                    if _host(root).tobytes() != wroot:
                        errors.append(f"thread {k} rep {rep} {job}: root differs from the oracle")
                if ctx.device_status() != 0:
                    errors.append(f"thread {k} rep {rep}: device status {ctx.device_status()}")
            ctx.close()
        except Exception as e:  # pragma: no cover
            errors.append(f"thread {k}: {e!r}")

    ts = [threading.Thread(target=worker, args=(k,)) for k in range(len(jobs))]
    for t in ts:
        t.start()
    for t in ts:
        t.join()
    assert not errors, errors
