"""world_size-2 gloo check of the benchmark's cross-rank plumbing (replicas only:
a barrier, a max of per-rank times, a sum of per-rank image counts)."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_shard_images_covers_every_image_once():
    sys.path.insert(0, ROOT)
    from paper_1905_00571_b200.dist import shard_images
    for total in (1, 7, 8, 129):
        for world in (1, 2, 3, 8):
            seen = []
            for r in range(world):
                first, count = shard_images(total, r, world)
                seen += list(range(first, first + count))
            assert seen == list(range(total))


def test_two_rank_gloo_max_and_sum(tmp_path):
    script = tmp_path / "w.py"
    script.write_text(textwrap.dedent("""
        import sys
        sys.path.insert(0, %r)
        from paper_1905_00571_b200 import dist
        rank, world, local = dist.init("gloo")
        dist.barrier()
        m = dist.max_over_ranks(1.5 + rank)
        s = dist.sum_over_ranks(10 + rank)
        assert world == 2 and m == 2.5 and s == 21.0, (world, m, s)
        dist.finalize()
        print("rank", rank, "ok")
    """ % ROOT))
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", "29611", str(script)]
    out = subprocess.run(cmd, capture_output=True, text=True, timeout=240)
    assert out.returncode == 0, out.stdout + out.stderr
    assert out.stdout.count("ok") == 2
