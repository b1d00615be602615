"""GPU parity for fbsr_round_desc (formats described at run time) against the oracle's descriptor path, and
against the built-in formats' kernels for the five built-in formats written as descriptors."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from helpers import VARIANTS, random_f32  # noqa: E402

# (K, P, B, max_code, inf_code, nan_code, single_zero)
BUILTIN = {
    "bf16": (16, 8, 127, 0x7F7F, 0x7F80, 0x7FC0, False),
    "fp16": (16, 11, 15, 0x7BFF, 0x7C00, 0x7E00, False),
    "e4m3": (8, 4, 7, 0x7E, None, 0x7F, False),
    "e5m2": (8, 3, 15, 0x7B, 0x7C, 0x7F, False),
    "b8p4": (8, 4, 8, 0x7E, 0x7F, 0x80, True),
}
OTHERS = {
    "e4m3fnuz": (8, 4, 8, 0x7F, None, 0x80, True),
    "e5m2fnuz": (8, 3, 16, 0x7F, None, 0x80, True),
    "b8p5": (8, 5, 4, 0x7E, 0x7F, 0x80, True),
    "e2m5": (8, 6, 2, 0x5F, None, 0x7F, False),
    "p13": (16, 13, 4, 0x7FFE, None, 0x8000, True),
    "wide": (16, 5, 127, 0x0FEF, 0x0FF0, 0x0FF8, False),
}


def setup_module(module):
    import paper_2504_20634_b200 as fbsr
    from oracle import capi
    import gpu_util
    module.fbsr, module.capi, module.gu = fbsr, capi, gpu_util


def inputs(args, n, seed):
    """Patterns over the format's whole range (below its smallest subnormal to beyond M) plus specials."""
    K, P, B, max_code = args[:4]
    rng = np.random.default_rng(seed)
    emax = (max_code >> (P - 1)) - B
    lo, hi = max(-126, 2 - P - B - 4), min(127, emax + 3)
    pats = random_f32(rng, n, lo, hi)
    from helpers import edge_values_f32
    edges = edge_values_f32()
    pats[rng.choice(n, size=edges.size, replace=False)] = edges
    return pats.view(np.float32)


@pytest.mark.parametrize("name", sorted(BUILTIN))
def test_builtin_formats_as_descriptors_equal_the_builtin_kernels(name):
    desc = fbsr.format_desc(*BUILTIN[name])
    assert fbsr.fbsr_format_desc_valid(desc)
    n = 50_000 + 3
    x = inputs(BUILTIN[name], n, 5)
    xd = torch.from_numpy(x).cuda()
    for variant in VARIANTS + ("rtne", "rta", "rto"):
        for k in (1, 2, 3, 5, 8, 11, 16):
            for ieee in (False, True):
                got = fbsr.fbsr_round_desc(xd, desc, variant, k, seed=21, offset=13, scale=0.8, ovf_ieee=ieee)
                ref = fbsr.fbsr_round(xd, name + ("+ieee" if ieee else ""), variant, k, seed=21, offset=13, scale=0.8)
                assert torch.equal(got, ref), (name, variant, k, ieee)
    od = capi.make_desc(*BUILTIN[name])
    gu.assert_codes_equal(fbsr.fbsr_round_desc(xd, desc, "src", 4, seed=2), capi.fbsr_round_desc(x, od, "src", 4, seed=2), name)


@pytest.mark.parametrize("name", sorted(OTHERS))
def test_other_formats_against_the_oracle(name):
    desc, od = fbsr.format_desc(*OTHERS[name]), capi.make_desc(*OTHERS[name])
    assert fbsr.fbsr_format_desc_valid(desc) and capi.desc_valid(od)
    dt = torch.uint16 if OTHERS[name][0] == 16 else torch.uint8
    n = 40_000 + 5
    x = inputs(OTHERS[name], n, 9)
    xd = torch.from_numpy(x).cuda()
    for variant in VARIANTS + ("rtne", "rta", "rto"):
        for k in range(1, 17):
            ieee = bool(k & 1)
            raw, out = gu.guarded(n, dt)
            fbsr.fbsr_round_desc(xd, desc, variant, k, seed=k, offset=7 * k, scale=1.25, ovf_ieee=ieee, out=out)
            torch.cuda.synchronize()
            expect = capi.fbsr_round_desc(x, od, variant, k, seed=k, offset=7 * k, scale=1.25, ieee_overflow=ieee)
            gu.assert_codes_equal(out, expect, "%s %s k=%d" % (name, variant, k))
            assert gu.canaries_intact(raw, n, dt)


def test_alignment_offsets_sizes_and_sharding():
    args = OTHERS["e4m3fnuz"]
    desc, od = fbsr.format_desc(*args), capi.make_desc(*args)
    x = inputs(args, 9000, 3)
    xd = torch.from_numpy(x).cuda()
    for n in (0, 1, 7, 8, 9, 255, 4099):
        for skip_in, skip_out in ((0, 0), (1, 0), (0, 3), (5, 1)):
            for offset in (0, 5, 2 ** 40 + 9):
                raw, out = gu.guarded(n, torch.uint8, misalign=skip_out)
                fbsr.fbsr_round_desc(xd[skip_in:skip_in + n], desc, "srf", 3, seed=6, offset=offset, out=out)
                torch.cuda.synchronize()
                gu.assert_codes_equal(out, capi.fbsr_round_desc(x[skip_in:skip_in + n], od, "srf", 3, seed=6, offset=offset),
                                      "n=%d skips %d/%d offset=%d" % (n, skip_in, skip_out, offset))
                assert gu.canaries_intact(raw, n, torch.uint8, misalign=skip_out)
    whole = fbsr.fbsr_round_desc(xd, desc, "src", 5, seed=1)
    cuts = [0, 3, 1000, 4097, 9000]
    parts = [fbsr.fbsr_round_desc(xd[a:b], desc, "src", 5, seed=1, offset=a) for a, b in zip(cuts[:-1], cuts[1:])]
    assert torch.equal(whole, torch.cat(parts))


def test_full_size_launch_and_torch_fnuz_cast():
    """2^27 elements in one launch: sampled slices against the oracle; round-to-nearest-even equals torch's own
    cast to float8_e4m3fnuz on every element with |y| <= M."""
    args = OTHERS["e4m3fnuz"]
    desc, od = fbsr.format_desc(*args), capi.make_desc(*args)
    n = 1 << 27
    g = torch.Generator(device="cuda").manual_seed(17)
    x = torch.randn(n, device="cuda", generator=g) * 30.0
    got = fbsr.fbsr_round_desc(x, desc, "srf", 3, seed=4)
    for a in (0, 12345 * 8, n - 4096):
        gu.assert_codes_equal(got[a:a + 4096], capi.fbsr_round_desc(x[a:a + 4096].cpu().numpy(), od, "srf", 3, seed=4, offset=a),
                              "slice %d" % a)
    rt = fbsr.fbsr_round_desc(x, desc, "rtne", 1, seed=0)
    inside = x.abs() <= 240.0
    assert torch.equal(rt[inside], x.to(torch.float8_e4m3fnuz).view(torch.uint8)[inside])


def test_rejected_descriptors_and_arguments():
    x = torch.zeros(64, device="cuda")
    for bad in ((12, 4, 7, 0x7E, None, 0x7F, False), (8, 1, 7, 0x7E, None, 0x7F, False), (16, 14, 7, 0x7E, None, 0x7FFF, False),
                (8, 4, 0, 0x7E, None, 0x7F, False), (8, 4, 7, 0x7E, 0x7E, 0x7F, False), (8, 4, 7, 0x7E, None, 0x7F, True)):
        desc = fbsr.format_desc(*bad)
        assert not fbsr.fbsr_format_desc_valid(desc)
        with pytest.raises(fbsr.FbsrError) as err:
            fbsr.fbsr_round_desc(x, desc, "srf", 3, seed=0, out=torch.empty(64, dtype=torch.uint16 if bad[0] == 16 else torch.uint8, device="cuda"))
        assert err.value.status == 1
    good = fbsr.format_desc(*OTHERS["b8p5"])
    for kw in (dict(k_bits=0), dict(k_bits=17), dict(scale=0.0)):
        a = dict(k_bits=3, scale=1.0)
        a.update(kw)
        with pytest.raises(fbsr.FbsrError):
            fbsr.fbsr_round_desc(x, good, "srf", a["k_bits"], seed=0, scale=a["scale"])
