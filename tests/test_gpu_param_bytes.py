"""sb_param_bytes through the C ABI against the arithmetic of the paper's Table 1 (Evaluation: the VGG variant
with 7 conv and 3 FC layers): what one worker of an MP group of size K holds is every conv parameter plus one
1/K column shard of every FC layer.  For K = 8 that is a saving of 65.8 % of the 6,990,666 parameters."""
import os

import pytest

import sb_inputs as si

pytestmark = pytest.mark.gpu

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "table1_vgg_variant_params.txt")


def table1():
    conv = fc = 0
    rows = []
    for line in open(GOLDEN):
        f = line.split()
        if not f or f[0].startswith("#") or f[0].startswith("share"):
            continue
        name, n_in, n_out, n_w = f[0], int(f[1]), int(f[2]), int(f[3])
        rows.append((name, n_in, n_out, n_w))
        if name.startswith("Conv"):
            conv += n_w + n_out          # weights + one bias per output channel
        else:
            fc += n_w + n_out
    return rows, conv, fc


@pytest.mark.parametrize("K", [1, 2, 4, 8])
def test_param_bytes_per_worker_match_table1(K):
    from paper_2112_15317_b200 import binding as sb
    rows, conv, fc = table1()
    assert conv + fc == 6990666
    wl = si.config(5).with_partition(1, K)        # Table 1's network; one replica of 128 images, K shards
    m = sb.Model.from_workload(wl, precision=sb.SB_FP32)
    per_shard = [m.param_bytes(j) for j in range(K)]
    m.close()
    # every worker: all conv parameters + its column shard of each FC layer (FC2's 10 columns split unevenly)
    for j, got in enumerate(per_shard):
        want = conv
        for name, n_in, n_out, _ in rows:
            if name.startswith("FC"):
                cols = si.shard_bounds(n_out, K)[j + 1] - si.shard_bounds(n_out, K)[j]
                want += cols * (n_in + 1)
        assert got == 4 * want, (j, got, want)
    # summed over the group: the logical parameters once, plus K - 1 further copies of the replicated conv part
    assert sum(per_shard) == 4 * (conv + fc + (K - 1) * conv)
    if K == 8:
        for got in per_shard:
            assert round(100.0 * (1.0 - got / (4.0 * (conv + fc))), 1) == 65.8
    if K == 1:
        assert per_shard[0] == 4 * 6990666


def test_layers_kept_whole_are_counted_in_full_for_every_worker():
    """An FC layer that the partitioning keeps whole (SB_FC_RELU_WHOLE) is held in full by every worker."""
    from paper_2112_15317_b200 import binding as sb
    K = 4
    layers = [(si.CONV3X3_RELU, 16), (si.MAXPOOL2, 0), (si.FC_RELU_WHOLE, 48), (si.FC_RELU, 64), (si.FC, 12), (si.SOFTMAX_XENT, 12)]
    wl = si.Workload("whole", layers, 8, 8, 3, 2, 1, K)
    m = sb.Model.from_workload(wl, precision=sb.SB_FP32)
    conv = 16 * 27 + 16
    fc_whole = 48 * (4 * 4 * 16) + 48
    for j in range(K):
        want = conv + fc_whole + (64 // K) * (48 + 1) + (12 // K) * (64 + 1)
        assert m.param_bytes(j) == 4 * want
    m.close()
