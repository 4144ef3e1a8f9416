"""GPU test of dynakv_attend_rows_noalloc, the entry point for callers that cannot allocate device
memory (a serving stack that owns the whole device, a latency-critical section, a sandboxed
component).  Its output must equal that of the regular path: dynakv_decode_step with a token budget
that covers every cluster attends all rows, which is exactly what the no-alloc call computes.  The
library's scratch array is shared by all calls and keeps old contents, so the check is made on two
calls in a row with different queries.  This file is collected last on purpose."""
import numpy as np
import pytest
import torch

import oracle as O
import paper_2511_07427_b200 as P
from gen import CONFIGS, UnitStream, make_decode_chunk, make_prefill

pytestmark = pytest.mark.gpu

TOL_ABS, TOL_L2 = 2e-3, 1e-3     # the attention tolerances of the parity tests


def _reference_and_noalloc(cfg, n_units):
    streams = [UnitStream(cfg, u) for u in range(n_units)]
    K, V = make_prefill(streams)
    q, _, _ = make_decode_chunk(streams, 2)
    Kd, Vd, qd = K.cuda(), V.cuda(), q.cuda()
    ctx = P.DynaKV(P.DynaKVConfig(
        n_units=n_units, gqa_group=cfg.G, head_dim=cfg.d, kv_dtype=P.F32 if cfg.kv_dtype == "f32" else P.BF16,
        max_tokens=cfg.max_tokens, max_clusters=cfg.max_clusters, kmeans_iters=cfg.T,
        init_mode=P.INIT_RANDOM, assign_mode=1))
    ctx.build_index(Kd, Vd, cfg.M0, 11)
    out = torch.empty((n_units, cfg.G, cfg.d), dtype=torch.float32, device="cuda")   # caller-owned output, reused
    # the fp64 oracle's attention over all rows of unit 0 (one cluster holding everything), as a second reference
    o = O.OracleUnit(cfg.d, cfg.G, cfg.n_prefill, 1)
    o.install(K[0].double().numpy(), V[0].double().numpy(), np.zeros(cfg.n_prefill, np.int32), 1)
    for t in range(2):                                                              # two calls in a row
        ref = ctx.decode_step(qd[t], 10 ** 9).cpu().numpy().astype(np.float64)       # budget covers every cluster
        _, ntok = ctx.get_selection()
        assert int(ntok.min()) == cfg.n_prefill
        torch.cuda.synchronize()
        if t == 1:
            # the first call on a device looks the scratch array's address up; from then on a call must leave the
            # device's free memory and torch's allocator untouched
            free0, alloc0 = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated()
        P.attend_rows_noalloc(qd[t], Kd, Vd, out=out)
        torch.cuda.synchronize()
        if t == 1:
            assert torch.cuda.mem_get_info()[0] == free0 and torch.cuda.memory_allocated() == alloc0, \
                "dynakv_attend_rows_noalloc changed the device's free memory"
        got = out.cpu().numpy().astype(np.float64)
        err = np.abs(got - ref).max()
        l2 = np.linalg.norm(got - ref) / np.linalg.norm(ref)
        assert err <= TOL_ABS and l2 <= TOL_L2, f"call {t}: max abs {err:.3e}, relative L2 {l2:.3e}"
        want = o.attend(q[t, 0].double().numpy(), [0])
        err = np.abs(got[0] - want).max()
        l2 = np.linalg.norm(got[0] - want) / np.linalg.norm(want)
        assert err <= TOL_ABS and l2 <= TOL_L2, f"call {t} against the oracle: max abs {err:.3e}, relative L2 {l2:.3e}"
    ctx.destroy()


def test_noalloc_matches_decode_step_bf16():
    cfg = CONFIGS[2].scaled(n_prefill=777, steps=4, M0=20, max_clusters=64, T=3)
    _reference_and_noalloc(cfg, 5)


def test_noalloc_matches_decode_step_fp32_g3_d64():
    cfg = CONFIGS[1].scaled(Hq=3, Hkv=1, n_prefill=301, steps=4, M0=9, max_clusters=32, T=3)
    _reference_and_noalloc(cfg, 2)


def test_noalloc_rejects_more_units_than_the_scratch_holds():
    U, G, d = 127, 4, 128            # 127 * 16 * 4 * 130 floats > 4 MiB
    q = torch.zeros((U, G, d), device="cuda")
    K = torch.zeros((U, 4, d), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(P.DynaKVError, match="fixed scratch"):
        P.attend_rows_noalloc(q, K, K)
    out = P.attend_rows_noalloc(q[:126], K[:126], K[:126])      # the documented limit still runs
    assert float(out.abs().max()) == 0.0                         # zero values -> zero output
