"""The allocation-free loss entry point against the oracle and the regular one (collected last on purpose).

zipml_loss_codes_static serves callers that cannot let the library allocate device memory (no
cudaMalloc inside a latency-critical region, or under a pool that owns the GPU): its scratch is a
fixed array in the library image.  It must give the oracle's loss -- and so the same as zipml_loss(CODES)
-- also on a second call that finds the first call's leftovers in the shared scratch, and it must refuse
what does not fit or is misaligned, without launching anything.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_1611_05402_b200 import binding, synth

pytestmark = pytest.mark.gpu


def test_static_scratch_loss_matches_regular_entry_point_twice_in_a_row():
    from paper_1611_05402_b200.build import build
    build()
    dev = torch.device("cuda", 0)
    with binding.Context(dev) as ctx:
        results = []
        # two different problems back to back: the second call sees the first one's scratch contents
        for key, m, n, bits in (("c2", 3000, 1000, 8), ("c4", 2500, 300, 3)):
            w, A, b, xs = synth.make(key, m=m, n=n, device=dev)
            levels = ctx.zipml_optimal_levels(A, bits, 256) if key == "c4" else None
            ds = ctx.zipml_quantize(A, bits, seed=3, levels=levels,
                                    level_mode=binding.LEVELS_TABLE if levels is not None else binding.LEVELS_UNIFORM)
            x = (xs * 0.8).contiguous()
            want = ctx.zipml_loss(binding.LOSS_CODES, b, x, data=ds)
            ctx.zipml_sync()
            # the oracle's estimate from the very planes the kernels read
            ods = oracle.Dataset(ds.plane1.cpu().numpy(), ds.plane2.cpu().numpy(), m, n, bits,
                                 oracle.TABLE if levels is not None else oracle.UNIFORM, ds.feat_lo.cpu().numpy(),
                                 ds.feat_step.cpu().numpy() if ds.feat_step is not None else np.zeros(n, np.float32),
                                 levels.cpu().numpy() if levels is not None else None)
            want_oracle = oracle.loss_codes(ods, b.cpu().numpy(), x.cpu().numpy())
            out1 = torch.empty(1, dtype=torch.float64, device=dev)
            out2 = torch.empty(1, dtype=torch.float64, device=dev)
            # the first call on a device looks up the scratch address and loads the kernels; the second
            # call is watched at the driver level (torch's own counters do not see a cudaMalloc
            # made inside the library): the device's free memory must not shrink
            got = binding.zipml_loss_codes_static(ds, b, x, out=out1)
            torch.cuda.synchronize(dev)
            free_before = torch.cuda.mem_get_info(dev)[0]
            again = binding.zipml_loss_codes_static(ds, b, x, out=out2)
            torch.cuda.synchronize(dev)
            assert free_before - torch.cuda.mem_get_info(dev)[0] < (1 << 20)
            results.append((want.item(), got.item(), again.item(), want_oracle))
        for want, got, again, want_oracle in results:
            assert abs(got - want_oracle) <= 1e-6 * abs(want_oracle)   # the tolerance of the other loss tests
            assert abs(got - want) <= 1e-6 * abs(want)
            assert again == got                                  # same scratch, same order: bit-identical
        # a problem beyond the fixed scratch is refused, not truncated
        n_big = (1 << 18) + 64
        p = torch.zeros((2, binding.lib().zipml_row_bytes(n_big, 2)), dtype=torch.uint8, device=dev)
        big = binding.Dataset(p, p, 2, n_big, 2, binding.LEVELS_UNIFORM, torch.zeros(n_big, device=dev),
                              torch.zeros(n_big, device=dev), None)
        with pytest.raises(binding.ZipmlError) as e:
            binding.zipml_loss_codes_static(big, torch.zeros(2, device=dev), torch.zeros(n_big, device=dev))
        assert e.value.code == binding.ERR_WORKSPACE
        # a plane that is not 16-byte aligned is refused like everywhere else (the kernels load whole words)
        raw = torch.zeros(2 * 64 + 16, dtype=torch.uint8, device=dev)
        odd = raw[4: 4 + 128].view(2, 64)
        bad = binding.Dataset(odd, odd, 2, 100, 4, binding.LEVELS_UNIFORM, torch.zeros(100, device=dev),
                              torch.zeros(100, device=dev), None)
        with pytest.raises(binding.ZipmlError) as e:
            binding.zipml_loss_codes_static(bad, torch.zeros(2, device=dev), torch.zeros(100, device=dev))
        assert e.value.code == binding.ERR_INVALID_ARG
