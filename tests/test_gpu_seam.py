"""The Replicated -> Sharded seam across ranks as one kernel (Table 2: Gather forward, Scatter backward): two
processes on ONE GPU, rank 0 owning the LLM input sequence, rank 1 owning the encoder microbatch.  Rank 1's merge
kernel stores straight into rank 0's buffer through an IPC mapping and its reverse gathers the gradient rows from it.
No kernel of one process waits for a kernel of the other: the hand-over is a host-level barrier after a stream sync."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.multiprocessing as mp

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, n_llm, hidden, result_q):
    sys.path.insert(0, ROOT)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    import torch.distributed as dist
    import oracle
    from paper_2607_03229_b200 import binding as B, dist as D, workloads as W
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    torch.cuda.set_device(0)
    w = W.tiny()
    T = w.total_tokens
    emb_bits = W.normal_bf16(77, 0, (n_llm, hidden))
    enc_bits = W.normal_bf16(77, 1, (T, hidden))
    pos = w.positions
    try:
        if rank == 0:
            # the first stage owns the LLM input sequence: its own allocation (cudaMalloc, not a slice of torch's pool block)
            emb = torch.empty((max(n_llm * hidden, 1 << 20),), dtype=torch.bfloat16, device="cuda")[:n_llm * hidden].view(n_llm, hidden)
            emb.copy_(torch.from_numpy(emb_bits.view(np.int16)).view(torch.bfloat16))
            torch.cuda.synchronize()
        else:
            emb = None
        shared = D.share_rows(emb, src_rank=0)
        dist.barrier()
        if rank == 1:
            enc = torch.from_numpy(enc_bits.view(np.int16)).view(torch.bfloat16).cuda()
            pos_dev = torch.from_numpy(pos).cuda()
            B.merge_tokens_peer(enc, shared, pos_dev, B.TRAINED)          # Coll(Gather, (enc, llm), m) as one kernel
            torch.cuda.synchronize()
        dist.barrier()
        if rank == 0:
            got = emb.cpu().view(torch.int16).numpy().view(np.uint16)
            want = oracle.merge_tokens(enc_bits, emb_bits, pos)
            result_q.put(("gather", bool(np.array_equal(got, want))))
            # pretend the LLM backward wrote the gradient of its input sequence in place
        dist.barrier()
        if rank == 1:
            d_enc = torch.full((T, hidden), 9.0, dtype=torch.bfloat16, device="cuda")
            B.merge_tokens_bwd_peer(shared, d_enc, pos_dev, B.TRAINED)     # Coll(Scatter, (enc, llm), m)
            torch.cuda.synchronize()
            got = d_enc.cpu().view(torch.int16).numpy().view(np.uint16)
            want = oracle.merge_tokens_bwd(oracle.merge_tokens(enc_bits, emb_bits, pos), pos)
            result_q.put(("scatter", bool(np.array_equal(got, want))))
            shared.close()
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_gather_and_scatter_seam_through_peer_memory():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29600 + os.getpid() % 300
    procs = [ctx.Process(target=_worker, args=(r, 2, port, 512, 256, q)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(timeout=180)
    assert all(p.exitcode == 0 for p in procs), [p.exitcode for p in procs]
    results = dict(q.get(timeout=5) for _ in range(2))
    assert results == {"gather": True, "scatter": True}
