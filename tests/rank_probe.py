"""Child process of test_launcher_starts_gloo_ranks: one CPU rank that joins the gloo group described by its
environment and writes `rank world local_rank max-over-ranks` to <dir>/rank<r>.txt."""
import os
import sys

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))

from paper_2608_00916_b200 import dist as pdist  # noqa: E402


def main():
    out_dir = sys.argv[1]
    rank, world, local = (int(os.environ[k]) for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK"))
    if len(sys.argv) > 2 and sys.argv[2] == "fail-on-1" and rank == 1:
        raise SystemExit(3)  # fails before joining anything
    if len(sys.argv) > 2:
        return  # the surviving rank of the failure case does not wait for its peer
    pdist.init(world, rank, backend="gloo")
    pdist.barrier()
    slowest = pdist.max_over_ranks(10.0 * (rank + 1))
    with open(os.path.join(out_dir, f"rank{rank}.txt"), "w") as fh:
        fh.write(f"{rank} {world} {local} {slowest}")
    pdist.finish()


if __name__ == "__main__":
    main()
