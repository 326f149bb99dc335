"""4-bit and 3-bit round-to-nearest factors (App. "Integrate with Quantization") on the GPU: the quantiser's codes and
parameters against the oracle's bit for bit, the dequantised values bit for bit, and the decode step gathering from
the codes against the oracle run on the dequantised bases."""
import numpy as np
import pytest
import torch

from oracle import xkv_oracle as O
from paper_2503_18893_b200 import synth, workload
from tests import _cases as C

pytestmark = pytest.mark.gpu
TOL = 2e-2


def _unpack(codes_u8, cols):
    """Library code layout -> plain codes [rows][cols]: in every 32-bit word nibble k of the low half is e_2k and
    nibble k of the high half is e_2k+1."""
    w = codes_u8.reshape(-1, cols // 8, 4).astype(np.uint32)
    word = w[..., 0] | (w[..., 1] << 8) | (w[..., 2] << 16) | (w[..., 3] << 24)
    out = np.empty(word.shape + (8,), dtype=np.uint8)
    for e in range(8):
        out[..., e] = (word >> (4 * (e >> 1) + 16 * (e & 1))) & 15
    return out.reshape(-1, cols)


def _unpack3(rec_u8, cols):
    """3-bit records {meta, w0, w1, w2} per group of 32 -> (codes [rows][cols], scale, zero)."""
    w = rec_u8.reshape(-1, cols // 32, 4, 4).astype(np.uint32)
    word = w[..., 0] | (w[..., 1] << 8) | (w[..., 2] << 16) | (w[..., 3] << 24)          # (rows, groups, 4)
    codes = np.empty(word.shape[:2] + (32,), dtype=np.uint8)
    for e in range(30):
        j, k = e // 10, (e % 10) >> 1
        codes[..., e] = (word[..., 1 + j] >> (3 * k + 16 * (e & 1))) & 7
    for e, sh in ((30, 15), (31, 31)):
        codes[..., e] = ((word[..., 1] >> sh) & 1) | (((word[..., 2] >> sh) & 1) << 1) | (((word[..., 3] >> sh) & 1) << 2)
    scale, zero = _meta(word[..., 0].astype(np.int64))
    return codes.reshape(-1, cols), scale, zero


def _meta(meta_i32):
    m = meta_i32.astype(np.int64) & 0xffffffff
    scale = ((m & 0xffff) << 16).astype(np.uint32).view(np.float32)
    zero = (m & 0xffff0000).astype(np.uint32).view(np.float32)
    return scale, zero


@pytest.mark.parametrize("bits", [4, 3])
@pytest.mark.parametrize("rows,cols,amp", [(37, 64, 1.0), (256, 512, 3.0), (5, 1024, 0.01)])
def test_quantiser_and_dequantiser_bit_exact(rows, cols, amp, bits):
    from paper_2503_18893_b200 import xkv
    x = (synth.normal(synth.stream_key(77, rows, cols), (rows, cols)) * amp).to(torch.bfloat16)
    x[0, :32] = 0.5                                                      # a constant group: scale 0
    codes, meta = xkv.xkv_quantize_rtn(x.cuda(), bits)
    oc, osc, oz = O.rtn_quantize(C.f32(x), bits)
    torch.cuda.synchronize()
    if bits == 4:
        gc = _unpack(codes.cpu().numpy(), cols)
        gs, gz = _meta(meta.cpu().numpy().reshape(rows, cols // 32))
    else:
        assert meta is None
        gc, gs, gz = _unpack3(codes.cpu().numpy(), cols)
    assert np.array_equal(gc, oc)
    assert np.array_equal(gs, osc) and np.array_equal(gz, oz)
    xh = xkv.xkv_dequantize_rtn(codes, meta, bits)
    assert np.array_equal(C.f32(xh), O.rtn_dequantize(oc, osc, oz))


@pytest.mark.parametrize("bits", [4, 3])
@pytest.mark.parametrize("name,over", [
    ("d128_r64", dict(T=2048, k=256, d_h=128, r_k=64, r_v=64)),
    ("d64_r96_r160_rep7", dict(T=1024, k=128, H_kv=2, H_q=14, r_k=96, r_v=160)),       # odd slab counts: padding slabs
    ("d128_batch2_ragged", dict(T=1000, k=130, batch=2, d_h=128, r_k=128, r_v=64)),
])
def test_decode_step_from_quantised_bases(name, over, bits):
    from paper_2503_18893_b200 import xkv
    s = synth.config(1, **over)
    inp = C.case_from_factors(s)
    g = C.GpuCase(s, inp)
    ck, mk = xkv.xkv_quantize_rtn(g.inp.A_k, bits)
    cv, mv = xkv.xkv_quantize_rtn(g.inp.A_v, bits)
    xkv.xkv_group_set_quantized_bases(g.grp, ck, mk, cv, mv, bits)
    gidx, gcnt = g.select(0)                                             # the selection does not depend on the bases
    gout, glse = g.attend(gidx, gcnt, 0)
    assert g.status() == (0, 0)
    # the oracle on the dequantised bases (what the quantised cache stands for)
    deq = lambda a: torch.from_numpy(np.stack([O.rtn_dequantize(*O.rtn_quantize(C.f32(a[b]), bits)) for b in range(s.batch)])).to(torch.bfloat16)
    inp_q = workload.GroupInputs(deq(inp.A_k), deq(inp.A_v), inp.B_k, inp.B_v, inp.landmarks, inp.q)
    oidx, ocnt, oout, olse = C.oracle_step(s, inp_q, 0)
    np.testing.assert_array_equal(gidx, oidx)
    np.testing.assert_array_equal(gcnt, ocnt)
    assert C.rel_err(gout, oout) <= TOL, name
    np.testing.assert_allclose(glse, olse, atol=2e-2)
    # and it differs from the 16-bit result by the quantisation error, i.e. the codes were really used
    _, _, oout16, _ = C.oracle_step(s, inp, 0)
    assert C.rel_err(gout, oout16) > 2e-3
    # back to the 16-bit bases
    xkv.xkv_group_set_quantized_bases(g.grp, None, None, None, None)
    gout16, _ = g.attend(gidx, gcnt, 0)
    assert C.rel_err(gout16, oout16) <= TOL
    g.close()


def test_quantisation_argument_checks():
    from paper_2503_18893_b200 import xkv
    x = torch.zeros((4, 48), dtype=torch.bfloat16, device="cuda")       # 48 is not a multiple of 32
    with pytest.raises(xkv.XKVError) as e:
        xkv.xkv_quantize_rtn(x)
    assert e.value.status == xkv.XKV_ERR_INVALID_ARG
    with pytest.raises(xkv.XKVError) as e:
        xkv.xkv_quantize_rtn(torch.zeros((4, 64), dtype=torch.bfloat16, device="cuda"), bits=5)
    assert e.value.status == xkv.XKV_ERR_UNSUPPORTED
