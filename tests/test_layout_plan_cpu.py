"""The multi-tensor launch metadata as a pure host function (palsgd_plan_layout): which tensors fuse into
segments, the scalar head that puts a segment's buffers back on an aligned grid, the chunk count.  Addresses
are made up (nothing is dereferenced), so these run without a GPU."""
import numpy as np
import pytest

import paper_2504_18454_b200 as P

BASE = 0x7F0000000000          # a multiple of 2 MB, like a fresh device allocation


def _packed(numel, K, esize, base, shift=0, pitch=None):
    """K rows of a packed arena: row k starts at base + k * pitch bytes, tensors back to back, all shifted by
    `shift` elements."""
    tot = int(sum(numel))
    pitch = pitch if pitch is not None else (tot + shift + 255) // 256 * 256 * esize
    starts = np.concatenate([[0], np.cumsum(numel)])[:-1]
    return [[base + k * pitch + (shift + int(s)) * esize for s in starts] for k in range(K)]


def _plan(numel, K=4, precision=P.PREC_FP32, inner=P.INNER_ADAMW, shift=0, pitch_elems=None, bases=None, **over):
    pe = 2 if precision == P.PREC_BF16_MASTER else 4
    bases = bases or {}
    mk = lambda name, i, K_, es: _packed(numel, K_, es, bases.get(name, BASE + i * (1 << 32)), shift,
                                         None if pitch_elems is None else pitch_elems * es)
    args = dict(param=mk("param", 0, K, pe), grad=mk("grad", 1, K, pe), m=mk("m", 2, K, 4),
                global_=mk("global_", 4, 1, 4)[0], outer_mom=mk("outer_mom", 5, 1, 4)[0])
    if inner == P.INNER_ADAMW:
        args["v"] = mk("v", 3, K, 4)
    if precision == P.PREC_BF16_MASTER:
        args["master"] = mk("master", 6, K, 4)
    args.update(over)
    return P.plan_layout(K=K, numel=numel, precision=precision, inner=inner, **args)


def test_a_packed_aligned_list_is_one_segment_without_a_head():
    numel = [50257 * 8, 2048, 7, 0, 12]
    lay = _plan(numel)
    assert lay["segments"] == [(0, 5, 0)] and lay["chunk_elems"] == 4096          # fp32 AdamW: 4096-element chunks
    assert lay["n_chunks"] == -(-sum(numel) // 4096)
    lay = _plan(numel, inner=P.INNER_SGDM)
    assert lay["chunk_elems"] == 8192 and lay["n_chunks"] == -(-sum(numel) // 8192)


@pytest.mark.parametrize("precision", [P.PREC_FP32, P.PREC_BF16_MASTER])
@pytest.mark.parametrize("shift", [1, 2, 3, 100, 255, 256, 257])
def test_a_shifted_packed_list_gets_the_head_up_to_the_next_multiple_of_256_elements(shift, precision):
    numel = [100000, 33]
    lay = _plan(numel, shift=shift, precision=precision, inner=P.INNER_SGDM)
    head = (-shift) % 256
    assert lay["segments"] == [(0, 2, head)]
    assert lay["n_chunks"] == (1 if head else 0) + -(-(sum(numel) - head) // 8192)


def test_rows_that_are_not_a_multiple_of_the_grid_apart_settle_for_less():
    numel = [5000]
    # fp32 rows 128 elements (512 bytes) apart mod 1024: 1024-byte alignment in all rows is out of reach, 512 is not
    assert _plan(numel, shift=1, pitch_elems=5120 + 128)["segments"] == [(0, 1, 127)]
    # 64 elements (256 bytes): head up to the next 256-byte boundary
    assert _plan(numel, shift=1, pitch_elems=5120 + 64)["segments"] == [(0, 1, 63)]
    # 8 elements (32 bytes): only 16 bytes are common to all rows
    assert _plan(numel, shift=1, pitch_elems=5120 + 8)["segments"] == [(0, 1, 3)]
    assert _plan(numel, shift=0, pitch_elems=5120 + 8)["segments"] == [(0, 1, 0)]
    # one buffer kind off by two elements against the others: no head serves all of them beyond 16 bytes ... and with
    # an odd offset none at all, so the segment takes the scalar path
    assert _plan(numel, bases={"m": BASE + 2 * (1 << 32) + 16})["segments"] == [(0, 1, 0)]
    assert _plan(numel, bases={"m": BASE + 2 * (1 << 32) + 8})["segments"] == [(0, 1, -1)]


def test_bf16_buffers_count_in_elements_too():
    numel = [70000]
    lay = _plan(numel, precision=P.PREC_BF16_MASTER, shift=1)                    # bf16 at +2 bytes, fp32 at +4
    assert lay["segments"] == [(0, 1, 255)]
    # bf16 rows 128 elements (256 bytes) apart mod 512, fp32 rows 512 bytes apart mod 1024: the second level
    lay = _plan(numel, precision=P.PREC_BF16_MASTER, shift=1, pitch_elems=70144 + 128)
    assert lay["segments"] == [(0, 1, 127)]


def test_gaps_and_empty_tensors_cut_segments():
    numel = [1000, 0, 24, 3000]
    K = 2
    # one allocation per tensor: nothing is adjacent
    sep = lambda i, es: [[BASE + (i * 64 + k * 8 + j) * (1 << 20) for j in range(4)] for k in range(K)]
    args = dict(param=sep(0, 4), grad=sep(1, 4), m=sep(2, 4), v=sep(3, 4), global_=sep(4, 4)[0], outer_mom=sep(5, 4)[0])
    lay = P.plan_layout(K=K, numel=numel, **args)
    assert lay["segments"] == [(0, 1, 0), (2, 1, 0), (3, 1, 0)]                  # the empty tensor makes no segment
    assert lay["n_chunks"] == 3
    # packed, but the momentum buffer has a hole behind the first tensor
    packed = _plan(numel, K=K)
    assert packed["segments"] == [(0, 4, 0)]
    m = _packed(numel, K, 4, BASE + 2 * (1 << 32))
    for k in range(K):
        for j in range(1, 4):
            m[k][j] += 4096
    lay = _plan(numel, K=K, m=m)
    # (the second run starts 1000 elements into every row: 24 more reach the next multiple of 256)
    assert lay["segments"] == [(0, 1, 0), (1, 3, 24)]
    # a NULL pointer for the empty tensor (what an empty torch tensor reports) also ends the run
    g = _packed(numel, K, 4, BASE + (1 << 32))
    for k in range(K):
        g[k][1] = 0
    lay = _plan(numel, K=K, grad=g)
    assert [s[:2] for s in lay["segments"]] == [(0, 1), (2, 2)]


def test_argument_errors_are_those_of_init():
    numel = [100]
    with pytest.raises(P.PalsgdError) as e:
        _plan(numel, bases={"m": BASE + 2})                                      # not even element-aligned
    assert e.value.status == -2
    with pytest.raises(P.PalsgdError) as e:
        _plan(numel, K=0)
    assert e.value.status == -1
    bad = _packed(numel, 4, 4, BASE)
    bad[2][0] = 0
    with pytest.raises(P.PalsgdError) as e:
        _plan(numel, param=bad)                                                  # NULL for a non-empty tensor
    assert e.value.status == -1
    L = P.lib()
    assert L.palsgd_plan_layout(None, 1, None, None, None, None, None, None, None, None) == -1
