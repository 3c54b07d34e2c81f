"""zoa_onebit_allreduce_static: the 1-bit AllReduce for callers that may not
allocate device memory (code inside an allocator-managed region, latency-critical
loops that cannot take cudaMalloc's implicit synchronisation, pre-partitioned
multi-tenant processes, clean-up paths that run when the device is full).  Its
packed intermediate lives in an array built into the library, so a call makes no
allocation.  This test calls it through the C ABI twice in a row and checks the
results against the handle-based entry point (zoa_onebit_reduce), bit for bit,
and against the CPU oracle's Algorithm 3 within the tolerance of the parity tests.
It is collected last on purpose, and passes alone in a fresh process as well."""
import numpy as np
import pytest
import torch

from helpers import assert_close
from oracle import zoa_oracle as zo
from paper_2202_06009_b200 import Zoa, ZoaError, binding as B

pytestmark = pytest.mark.gpu


def _existing(z_rounds, n, W, chunk):
    """The same two rounds through a handle: u := z, then zoa_onebit_reduce."""
    out = []
    with Zoa(n, W, chunk=chunk) as h:
        for r, z in enumerate(z_rounds):
            for i in range(W):
                h.write("u", z[i], i)
            B.zoa_set_scalars(h.h, 1.0, 0, r)      # something was accumulated, so a sync is allowed
            h.onebit_reduce()
            torch.cuda.synchronize()
            bits = np.unpackbits(h.read("words_s").view(np.uint8), bitorder="little")[:n].astype(bool)
            scale = np.repeat(h.read("scales_s"), chunk)[:n]
            out.append({"z_bar": np.where(bits, scale, -scale).astype(np.float32),
                        "delta_w": np.stack([h.read("delta_w", i) for i in range(W)]),
                        "delta_s": h.read("delta_s")})
    return out


@pytest.mark.parametrize("n,W,chunk,offset", [(3 * 1024 + 77, 4, 1024, 0), (5000, 3, 256, 0), (4096 + 9, 2, 4096, 1)])
def test_static_entry_point_matches_the_handle_path_twice_in_a_row(n, W, chunk, offset):
    rng = np.random.default_rng(n + W)
    z_rounds = [rng.standard_normal((W, n)).astype(np.float32) * np.float32(1 + r) for r in range(2)]
    want = _existing(z_rounds, n, W, chunk)
    cpu = zo.Oracle(n, W, chunk, dtype=np.float32)       # Algorithm 3 with errors that start at zero

    # `offset` shifts every buffer by one float to exercise the unaligned path
    def dev(a):
        t = torch.zeros(a.size + offset, device="cuda")
        v = t[offset:]
        v.copy_(torch.from_numpy(np.ascontiguousarray(a)))
        return v

    delta_w = [dev(np.zeros(n, np.float32)) for _ in range(W)]
    delta_s, z_bar = dev(np.zeros(n, np.float32)), dev(np.zeros(n, np.float32))
    stream = torch.cuda.current_stream().cuda_stream
    for r in range(2):
        z = [dev(z_rounds[r][i]) for i in range(W)]
        B.zoa_onebit_allreduce_static([t.data_ptr() for t in z], [t.data_ptr() for t in delta_w],
                                      delta_s.data_ptr(), z_bar.data_ptr(), n, W, chunk, stream)
        torch.cuda.synchronize()
        z_bar_cpu = cpu.onebit_allreduce(z_rounds[r])
        assert_close(z_bar.cpu().numpy(), z_bar_cpu, f"z_bar against the oracle, call {r}")
        assert np.array_equal(z_bar.cpu().numpy() >= 0, z_bar_cpu >= 0), f"signs of z_bar against the oracle, call {r}"
        assert_close(delta_s.cpu().numpy(), cpu.delta_bar, f"delta_s against the oracle, call {r}")
        for i in range(W):
            assert_close(delta_w[i].cpu().numpy(), cpu.delta[i], f"delta_w[{i}] against the oracle, call {r}")
        assert np.array_equal(z_bar.cpu().numpy(), want[r]["z_bar"]), f"z_bar, call {r}"
        assert np.array_equal(delta_s.cpu().numpy(), want[r]["delta_s"]), f"delta_s, call {r}"
        for i in range(W):
            got = delta_w[i].cpu().numpy()
            assert np.all(np.abs(got - want[r]["delta_w"][i]) <= 1e-7 + 1e-5 * np.abs(want[r]["delta_w"][i]))
            assert np.array_equal(got, want[r]["delta_w"][i]), f"delta_w[{i}], call {r}"


def test_static_entry_point_rejects_what_does_not_fit():
    slots = B.zoa_static_scratch_slots()
    assert slots == 1 << 20
    t = torch.zeros(64, device="cuda")
    p = t.data_ptr()
    n_big = 32 * slots          # one worker's sign words alone fill the array; the magnitudes no longer fit
    with pytest.raises(ZoaError) as e:
        B.zoa_onebit_allreduce_static([p], [p], p, p, n_big, 1, 4096, 0)
    assert e.value.status == B.ERR_ARG and "scratch" in str(e.value)
    with pytest.raises(ZoaError):
        B.zoa_onebit_allreduce_static([p], [p], p, p, 64, 1, 48, 0)
    # sizes whose slot count would wrap 64-bit arithmetic are refused as arguments too, not at launch
    for n_huge, W, chunk in ((1 << 62, 64, 32), ((1 << 63) + 5, 1, 4096), (32 * slots + 1, 1, 16384)):
        with pytest.raises(ZoaError) as e:
            B.zoa_onebit_allreduce_static([p] * W, [p] * W, p, p, n_huge, W, chunk, 0)
        assert e.value.status == B.ERR_ARG
