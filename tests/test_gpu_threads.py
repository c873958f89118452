"""Several host threads make their FIRST calls into the library at the same time (a fresh process, so the
per-device one-time set-up of every launcher is raced), each on its own stream and its own buffers; every
result must equal the one the same call gives afterwards on a single thread."""
import subprocess
import sys
import textwrap

import pytest

pytestmark = pytest.mark.gpu

CHILD = textwrap.dedent('''
    import threading, sys
    import numpy as np, torch
    from paper_2609_35465_b200 import synth, tetra as tt
    sys.path.insert(0, "tests")
    from helpers import make_matrix

    torch.cuda.init()
    table = tt.tetra_build_table(synth.DEFAULT_GAIN)
    torch.cuda.synchronize()

    def upload(m):
        codes = torch.from_numpy(m["codes"]).cuda()
        d = dict(N=m["N"], K=m["K"], codes=tt.tetra_pack_codes(codes, table, m["N"], m["B"]),
                 row_scales=torch.from_numpy(m["sigma"]).cuda(), x=torch.from_numpy(m["x"]).cuda(),
                 tail=torch.from_numpy(m["tail"]).cuda() if m["tail"] is not None else None)
        d["y"] = torch.full((m["x"].shape[0], m["N"]), float("nan"), dtype=torch.float32, device="cuda")
        return d

    mats = [make_matrix(81, i, N, K, True, batch=b) for i, (N, K, b) in
            enumerate([(520, 2560, 1), (300, 24 * 65 + 8, 1), (256, 4096, 5), (264, 3080, 16), (96, 24 * 40, 1), (40, 24 * 700, 1)])]
    devs = [upload(m) for m in mats]
    w = torch.from_numpy(np.random.default_rng(5).standard_normal((4096, 24)).astype(np.float32)).cuda()
    torch.cuda.synchronize()

    def call(i, stream):
        d = devs[i]
        if i == 0:
            tt.tetra_gemv_tail(d["codes"], d["row_scales"], table, d["x"], d["y"], d["N"], d["K"], 1, d["tail"], stream=stream)
        elif i == 1:
            pr = tt.make_problems([d])
            ws = torch.empty(max(16, tt.tetra_grouped_workspace_bytes(pr)), dtype=torch.uint8, device="cuda")
            tt.tetra_gemv_grouped(pr, table, ws, stream=stream)
            d["ws"] = ws
        elif i in (2, 3):
            b = d["x"].shape[0]
            ws = torch.empty(tt.tetra_batched_workspace_bytes(d["N"], d["K"]), dtype=torch.uint8, device="cuda")
            tt.tetra_gemv_batched(d["codes"], d["row_scales"], table, d["x"], d["y"], d["N"], d["K"], b, d["tail"], ws, stream=stream)
            d["ws"] = ws
        elif i == 4:
            tt.tetra_gemv_list(tt.make_problems([d]), table, stream=stream)
        else:
            d["enc"] = tt.tetra_encode_blocks(w, table, stream=stream)

    def worker(i, barrier):
        s = torch.cuda.Stream()
        barrier.wait()
        for _ in range(3):
            call(i, s)
        s.synchronize()

    barrier = threading.Barrier(len(devs))
    threads = [threading.Thread(target=worker, args=(i, barrier)) for i in range(len(devs))]
    for t in threads: t.start()
    for t in threads: t.join()
    torch.cuda.synchronize()
    first = [d["y"].cpu().numpy().copy() for d in devs]
    enc_first = [t.cpu().numpy().copy() for t in devs[5]["enc"]]
    for i, d in enumerate(devs):
        d["y"].fill_(float("nan"))
        call(i, None)
    torch.cuda.synchronize()
    for i, d in enumerate(devs[:5]):
        y = d["y"].cpu().numpy()
        assert np.isfinite(y).all(), i
        assert np.array_equal(y, first[i]), "call %d differs between the threaded and the single-threaded run" % i
    for a, b in zip(enc_first, [t.cpu().numpy() for t in devs[5]["enc"]]):
        assert np.array_equal(a, b)
    print("THREADS-OK")
''')


def test_first_calls_from_several_threads_at_once():
    res = subprocess.run([sys.executable, "-c", CHILD], capture_output=True, text=True, timeout=600)
    assert res.returncode == 0, res.stdout[-2000:] + res.stderr[-4000:]
    assert "THREADS-OK" in res.stdout
