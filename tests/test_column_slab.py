"""Column-slab split of one equation over several devices: the library's slab bounds and descriptors against their
plain definitions, the identity X[:, b:e] = M1...M(n-1) Mn[:, b:e] + T[:, b:e] on the oracle, and the gather of the
slabs over two gloo ranks (each rank's slab comes from the oracle here: no GPU)."""
import os
import sys

import numpy as np
import pytest

torch = pytest.importorskip("torch")
import torch.distributed as dist
import torch.multiprocessing as mp

import paper_2208_10391_b200 as mom
import workloads as wl
from oracle import values as ov

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_slabs_partition_the_columns_evenly_in_whole_units():
    for multiple in (1, 4, 7):
        for cols in range(1, 70):
            for world in range(1, 10):
                bounds = [mom.mom_column_slab(cols, r, world, multiple) for r in range(world)]
                assert bounds[0][0] == 0 and bounds[-1][1] == cols
                for (b0, e0), (b1, e1) in zip(bounds[:-1], bounds[1:]):
                    assert e0 == b1                                     # contiguous, in rank order
                units = []
                for b, e in bounds:
                    assert b <= e and b % multiple == 0 and (e % multiple == 0 or e == cols)
                    units.append(-(-(e - b) // multiple))
                assert max(units) - min(units) <= 1, (cols, world, multiple, bounds)
    assert mom.mom_column_slab(8192, 3, 8) == (3072, 4096)
    assert mom.mom_column_slab(1 << 62, 1, 2, 4) == (1 << 61, 1 << 62)


def test_slab_errors():
    for args in ((0, 0, 1, 4), (8, -1, 2, 4), (8, 2, 2, 4), (8, 0, 0, 4), (8, 0, 1, 0)):
        with pytest.raises(mom.MomError) as e:
            mom.mom_column_slab(*args)
        assert e.value.status == mom.ERR_INVALID_ARG
    for args in (((8, 8, 0), False, -1, 4), ((8, 8, 0), False, 4, 4), ((8, 6, 0), False, 0, 7), ((8, 6, 0), True, 0, 9)):
        with pytest.raises(mom.MomError) as e:
            mom.mom_column_slab_desc(*args)
        assert e.value.status == mom.ERR_INVALID_ARG
    with pytest.raises(mom.MomError) as e:
        mom.mom_column_slab_desc((8, 6, mom.LOWER_TRI), False, 0, 2)
    assert e.value.status == mom.ERR_PROPERTY


def test_slab_descriptors():
    d = mom.mom_column_slab_desc((8, 6, mom.GENERAL), False, 2, 5)
    assert (d.rows, d.cols, d.property) == (8, 3, mom.GENERAL)
    d = mom.mom_column_slab_desc((8, 6, mom.GENERAL), True, 2, 5)         # used 6 x 8: columns 2..5 are stored rows 2..5
    assert (d.rows, d.cols, d.property) == (3, 6, mom.GENERAL)
    d = mom.mom_column_slab_desc((8, 8, mom.UPPER_TRI), False, 4, 8)      # a proper slab of a triangle is general
    assert (d.rows, d.cols, d.property) == (8, 4, mom.GENERAL)
    d = mom.mom_column_slab_desc((8, 8, mom.UPPER_TRI), False, 0, 8)      # the whole operand keeps its type
    assert (d.rows, d.cols, d.property) == (8, 8, mom.UPPER_TRI)
    assert mom.column_slab_equation([(8, 8, 1), (8, 2, 0)], [], 0, 3) is None     # two columns, three devices


def slab_arrays(eq, chain, add, begin, end):
    """This device's operands: the last factor and every Add term cut to columns [begin, end) as used."""
    def cut(a, desc, t):
        if a is None:                                   # Identity: the slab has to be stored
            a = np.eye(desc[0], dtype=np.float32)
        return np.ascontiguousarray(a[begin:end, :] if t else a[:, begin:end])
    ct = list(eq.chain_t) + [False] * (len(chain) - len(eq.chain_t))
    at = list(eq.add_t) + [False] * (len(add) - len(eq.add_t))
    whole = begin == 0 and end == (eq.descs()[-1][0] if ct[-1] else eq.descs()[-1][1])
    if whole:
        return list(chain), list(add)
    return list(chain[:-1]) + [cut(chain[-1], eq.descs()[-1], ct[-1])], [cut(a, d, t) for a, d, t in zip(add, eq.add_descs(), at)]


def oracle_slab(eq, chain, add, rank, world):
    got = mom.column_slab_equation(eq.descs(), eq.add_descs(), rank, world, eq.chain_t, eq.add_t)
    if got is None:
        return None, (0, 0)
    cd, ad, begin, end = got
    c, a = slab_arrays(eq, chain, add, begin, end)
    cd = [(d.rows, d.cols, d.property) for d in cd]
    ad = [(d.rows, d.cols, d.property) for d in ad]
    c, cd = ov.transposed_operands(c, cd, eq.chain_t)
    a, ad = ov.transposed_operands(a, ad, eq.add_t)
    x, _ = ov.evaluate(c, cd, a, ad)
    return x, (begin, end)


def whole_value(eq, chain, add):
    c, cd = ov.transposed_operands(chain, eq.descs(), eq.chain_t)
    a, ad = ov.transposed_operands(add, eq.add_descs(), eq.add_t)
    return ov.evaluate(c, cd, a, ad)


@pytest.mark.parametrize("world", [1, 2, 3, 8])
def test_slab_values_tile_the_whole_value(world):
    for seed in range(12):
        eq = wl.random_equation(700 + seed, max_len=4, max_dim=40, kinds=True)
        chain, add = wl.generate(eq)
        x_ref, den = whole_value(eq, chain, add)
        x = np.full_like(x_ref, np.nan)
        for rank in range(world):
            xs, (b, e) = oracle_slab(eq, chain, add, rank, world)
            if xs is not None:
                x[:, b:e] = xs
        assert ov.normwise_error(x, x_ref, den) <= 1e-14


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import test_column_slab as me
    worst = 0.0
    for seed, cols_multiple in ((1, 4), (2, 4), (3, 1)):
        eq = wl.Equation(f"slab_{seed}", 900 + seed, (wl.Operand(24, 24, wl.LOWER_TRI), wl.Operand(24, 36, wl.GENERAL),
                                                    wl.Operand(36, 10 + 9 * seed, wl.GENERAL)),
                         (wl.Operand(24, 10 + 9 * seed, wl.GENERAL),))
        chain, add = wl.generate(eq)
        xs, (b, e) = me.oracle_slab(eq, chain, add, rank, world)
        rows, cols = 24, 10 + 9 * seed
        mine = torch.from_numpy(xs) if xs is not None else torch.empty((rows, 0), dtype=torch.float64)
        x = mom.gather_column_slabs(mine, rows, cols, rank, world)
        x_ref, den = me.whole_value(eq, chain, add)
        worst = max(worst, ov.normwise_error(x.numpy(), x_ref, den))
    out.put((rank, worst))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_gather_their_slabs_into_the_whole_result():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 31500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    results = sorted(q.get(timeout=180) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r for r, _ in results] == [0, 1]
    assert all(err <= 1e-14 for _, err in results)
