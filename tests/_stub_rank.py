"""One rank of the launcher test: joins the group the launcher prepared (gloo, CPU), pretends to have timed a
region, and rank 0 writes what the bench would compute from it."""
import json
import os
import sys

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))

from paper_2605_29986_b200 import rows  # noqa: E402


def main():
    rank, local_rank, world, dist = rows.init_ranks("gloo")
    assert world == 2 and dist is not None and local_rank == rank
    dist.barrier()
    slowest = rows.max_over_ranks(0.5 + rank, dist)     # rank r "took" 0.5 + r seconds
    spans = [list(rows.shard_rows(7, r, world)) for r in range(world)]
    dist.barrier()
    dist.destroy_process_group()
    if rank == 0:
        open(sys.argv[1], "w").write(json.dumps({"n_gpus": world, "seconds": slowest, "rows": spans}))


if __name__ == "__main__":
    main()
