"""Row sharding: host logic and a world_size-2 gloo run on CPU.

The shards are computed by the oracle here (no GPU in this test); what is checked is the sharding
contract itself: contiguous row blocks, `row_base` in the random-number counter, all_gather of the
per-row outputs, and that the assembled result equals the unsharded one."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, "tests"))

from paper_2502_01662_b200 import sharding, synth  # noqa: E402


def test_shard_rows_partition():
    for batch in (0, 1, 7, 8, 64, 257):
        for world in (1, 2, 3, 8):
            seen = []
            for r in range(world):
                first, count = sharding.shard_rows(batch, world, r)
                seen.extend(range(first, first + count))
            assert seen == list(range(batch))
            sizes = [sharding.shard_rows(batch, world, r)[1] for r in range(world)]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        sharding.shard_rows(4, 2, 2)


def _worker(rank, world, port, result_path):
    import helpers
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = synth.CONFIGS["cfg4"].scaled(batch=5, vocab=640, gamma=3, name="shard_case")
        inputs = synth.make_inputs(w, "cpu")            # same seed on every rank: same full batch
        first, count = sharding.shard_rows(w.batch, world, rank)
        ws = w.scaled(batch=count, name="shard")
        part = dict(inputs, logits=inputs["logits"][:, first:first + count].contiguous(),
                    drafts=inputs["drafts"][first:first + count].contiguous(),
                    proposer=inputs["proposer"][first:first + count].contiguous())
        got = helpers.run_oracle(ws, part, row_base=first)
        local = {k: torch.as_tensor(np.asarray(got[k]).astype(np.int64)) for k in ("accept_count", "out_tokens", "row_status")}
        full = sharding.gather_rows(local, w.batch)
        if rank == 0:
            ref = helpers.run_oracle(w, inputs)
            ok = all(np.array_equal(full[k].numpy(), np.asarray(ref[k]).astype(np.int64)) for k in local)
            with open(result_path, "w") as f:
                f.write("ok" if ok else "mismatch")
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_rank_gloo_shards_match_unsharded(tmp_path):
    port = 29500 + (os.getpid() % 2000)
    result = tmp_path / "result.txt"
    mp.spawn(_worker, args=(2, port, str(result)), nprocs=2, join=True)
    assert result.read_text() == "ok"
