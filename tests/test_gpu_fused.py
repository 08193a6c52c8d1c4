"""Decode fused into a bf16 matrix product (Section I, Section III-C: weights are decompressed
just before the computation that uses them) against the oracle: W is decoded and dequantised by
the ORACLE, the product is taken in float64 on the host, and the GPU's fp32-accumulated result
must agree within the bound of fp32 accumulation over K terms."""
import numpy as np
import pytest
import torch

import oracle
import synthgen as sg
import paper_2406_06237_b200 as ans
from paper_2406_06237_b200.runtime import DeviceBatch, pack_gemm_layer
from helpers import oracle_pack_spec, to_packed_layer

pytestmark = pytest.mark.gpu


def _bf16_bits_to_f64(bits):
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def _block_order():
    """Where element (r, c) of a 64 x 64 block lies among the block's 4096 symbols."""
    r, c = np.meshgrid(np.arange(64), np.arange(64), indexing="ij")
    return (r // 8) * 512 + (r % 8) * 64 + ((c // 8) ^ (r % 8)) * 8 + c % 8


def _blocked(w):
    """N x K -> the order the fused call wants: blocks of 64 x 64, [N/64][K/64][4096], each block
    in the tensor core's operand order."""
    n, k = w.shape
    blocks = w.reshape(n // 64, 64, k // 64, 64).transpose(0, 2, 1, 3).reshape(n // 64, k // 64, 4096)
    out = np.empty_like(blocks)
    out[:, :, _block_order().ravel()] = blocks
    return out.ravel()


def _unblocked(flat, n, k):
    """The inverse of _blocked."""
    blocks = flat.reshape(n // 64, k // 64, 4096)[:, :, _block_order().ravel()]
    return blocks.reshape(n // 64, k // 64, 64, 64).transpose(0, 2, 1, 3).reshape(n, k)


def _case(M, N, K, b, pzp, R, seed, scale=0.03125, quiet_rows=0):
    A, zp = sg.alphabet_for_bits(b)
    spec = sg.LayerSpec(f"w{N}x{K}", (N, K), b, A, zp, sg.theta_for_pzp(A, zp, pzp), scale, R, 4096, "bf16",
                        sg.stream_key(31, seed))
    w_sym = sg.draw_symbols(spec).reshape(N, K)
    if quiet_rows:                          # only every quiet_rows-th block row keeps its weights: sub-streams of very unequal length
        keep = (np.arange(N) // 64) % quiet_rows == 0
        w_sym[~keep] = zp
    T, P, f256 = oracle_pack_spec(spec, _blocked(w_sym), oracle.STRIPS, 32)
    dec, rc = oracle.unpack(T, P)
    assert rc == oracle.OK
    w_bits = oracle.dequant(dec, zp, scale, "bf16")           # blocked order
    w = _unblocked(_bf16_bits_to_f64(w_bits), N, K)
    assert (_unblocked(_blocked(w_sym), N, K) == w_sym).all()
    rng = np.random.default_rng(seed)
    x = torch.from_numpy(rng.standard_normal((M, K)).astype(np.float32)).to(torch.bfloat16)
    x64 = x.to(torch.float32).numpy().astype(np.float64)
    return spec, P, f256, x, x64, w


@pytest.mark.parametrize("M,N,K,b,pzp,R", [(128, 64, 64, 3, 0.7, 8), (128, 128, 256, 4, 0.6, 8), (1, 64, 128, 2, 0.9, 6),
                                           (77, 192, 320, 5, 0.85, 10), (128, 512, 1024, 3, 0.7, 12),
                                           (16, 64, 2048, 8, 0.9, 8)])
def test_fused_product_equals_the_oracles_weights_times_x(M, N, K, b, pzp, R):
    spec, P, f256, x, x64, w = _case(M, N, K, b, pzp, R, seed=M + N + K)
    db = DeviceBatch([to_packed_layer(spec, P, f256)])         # the table and the compressed bytes on the device
    xd = x.cuda()
    y = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    guard = torch.full((4096,), 7.0, dtype=torch.float32, device="cuda")
    ans.ans_decode_gemm_bf16(db.h_descs[0][0], xd.data_ptr(), M, N, K, y.data_ptr(), db.status.data_ptr(),
                             torch.cuda.current_stream().cuda_stream)
    assert db.read_status() == 0
    got = y.cpu().numpy().astype(np.float64)
    want = x64 @ w.T
    # products of two bf16 values are exact in fp32; the sums over K terms are rounded to fp32
    bound = (np.abs(x64) @ np.abs(w).T) * (K * 2.0 ** -24) + 1e-30
    assert np.isfinite(got).all() and (np.abs(got - want) <= bound).all(), float(np.abs(got - want).max())
    assert (guard == 7.0).all()


# The wide form of the kernel (tables of up to 256 states, N a multiple of 256): ranges that end
# inside the K steps of their 256 features (partial sums added in Y) and ranges that do not (plain
# stores: one unit per CTA with K = 64, or 37888 = 148 * 256 features with two steps each on a
# 148-SM part), several segments per CTA, stages reused many times, M below a full tile; and the
# forms with the operands exchanged that M <= 16 and M <= 32 take (Y^T = W X^T).
@pytest.mark.parametrize("M,N,K,b,pzp,R,quiet", [(128, 256, 256, 3, 0.7, 8, 0), (50, 512, 1024, 4, 0.6, 8, 0),
                                                 (128, 2048, 4800, 3, 0.8, 8, 0), (8, 19200, 640, 2, 0.9, 6, 0),
                                                 (33, 256, 64, 3, 0.7, 7, 0), (128, 1024, 2048, 6, 0.5, 8, 3),
                                                 (64, 256, 19008, 3, 0.7, 8, 0), (4, 19200, 1408, 3, 0.7, 8, 0),
                                                 (16, 37888, 128, 3, 0.7, 8, 0), (128, 1024, 64, 4, 0.6, 8, 0),
                                                 (32, 512, 1024, 3, 0.7, 8, 0), (17, 256, 2112, 4, 0.8, 8, 0),
                                                 (31, 2048, 4800, 3, 0.8, 7, 0), (1, 256, 256, 3, 0.7, 8, 0),
                                                 (12, 1024, 2048, 6, 0.5, 8, 3), (24, 19200, 640, 2, 0.9, 6, 0)])
def test_wide_form_equals_the_oracles_weights_times_x(M, N, K, b, pzp, R, quiet):
    spec, P, f256, x, x64, w = _case(M, N, K, b, pzp, R, seed=M + N + K, quiet_rows=quiet)
    if quiet:                               # the kept block rows' sub-streams are far above the average: they do not fit the staging room
        ext = np.diff(P.sub_offsets.astype(np.int64))
        assert ext.max() > 1.25 * ext.mean() + 512
    db = DeviceBatch([to_packed_layer(spec, P, f256)])
    xd = x.cuda()
    y = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    guard = torch.full((4096,), 7.0, dtype=torch.float32, device="cuda")
    st = torch.cuda.current_stream().cuda_stream
    for _ in range(2):                      # twice: the second call must not add to the first call's sums
        ans.ans_decode_gemm_bf16(db.h_descs[0][0], xd.data_ptr(), M, N, K, y.data_ptr(), db.status.data_ptr(), st)
    assert db.read_status() == 0
    got = y.cpu().numpy().astype(np.float64)
    want = x64 @ w.T
    bound = (np.abs(x64) @ np.abs(w).T) * ((K + 64) * 2.0 ** -24) + 1e-30
    assert np.isfinite(got).all() and (np.abs(got - want) <= bound).all(), float(np.abs(got - want).max())
    assert (guard == 7.0).all()


def test_the_librarys_own_packer_feeds_the_fused_call():
    """pack_gemm_layer (blocks in the operand's order, library encoder) -> fused call, against the
    weights dequantised by the oracle from the symbols as drawn."""
    M, N, K, b, R = 40, 512, 384, 3, 8
    A, zp = sg.alphabet_for_bits(b)
    spec = sg.LayerSpec("w", (N, K), b, A, zp, sg.theta_for_pzp(A, zp, 0.7), 0.0625, R, 4096, "bf16", sg.stream_key(31, 77))
    w_sym = sg.draw_symbols(spec).reshape(N, K)
    pl = pack_gemm_layer(w_sym, A, R, b, zp, 0.0625)
    w = _bf16_bits_to_f64(oracle.dequant(w_sym.ravel(), zp, 0.0625, "bf16")).reshape(N, K)
    x = torch.from_numpy(np.random.default_rng(3).standard_normal((M, K)).astype(np.float32)).to(torch.bfloat16)
    x64 = x.to(torch.float32).numpy().astype(np.float64)
    db = DeviceBatch([pl])
    y = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    ans.ans_decode_gemm_bf16(db.h_descs[0][0], x.cuda().data_ptr(), M, N, K, y.data_ptr(), db.status.data_ptr(),
                             torch.cuda.current_stream().cuda_stream)
    assert db.read_status() == 0
    got = y.cpu().numpy().astype(np.float64)
    bound = (np.abs(x64) @ np.abs(w).T) * ((K + 64) * 2.0 ** -24) + 1e-30
    assert (np.abs(got - x64 @ w.T) <= bound).all()


def test_wide_form_flags_a_corrupt_block():
    spec, P, f256, x, x64, w = _case(32, 256, 256, 3, 0.7, 8, seed=6)
    for where in (100, 3):                  # inside a lane's bits; inside the lengths that head the sub-stream
        s = P.stream.copy()
        s[int(P.sub_offsets[5]) + where] ^= 0x55
        P2 = oracle.Packed(P.layout, s, P.sub_offsets, P.lane_meta, P.n, P.chunk, P.groups)
        assert oracle.unpack(oracle.Table(f256[:spec.alphabet], 8), P2)[1] == oracle.ERR_CORRUPT
        db = DeviceBatch([to_packed_layer(spec, P2, f256)])
        y = torch.zeros((32, 256), dtype=torch.float32, device="cuda")
        ans.ans_decode_gemm_bf16(db.h_descs[0][0], x.cuda().data_ptr(), 32, 256, 256, y.data_ptr(), db.status.data_ptr(),
                                 torch.cuda.current_stream().cuda_stream)
        assert db.read_status() != 0
        assert torch.isfinite(y).all()


def test_fused_call_flags_a_corrupt_block_and_refuses_what_it_does_not_support():
    spec, P, f256, x, x64, w = _case(32, 128, 128, 3, 0.7, 8, seed=5)
    s = P.stream.copy()
    s[int(P.sub_offsets[2]) + 100] ^= 0x55
    P2 = oracle.Packed(P.layout, s, P.sub_offsets, P.lane_meta, P.n, P.chunk, P.groups)
    T = oracle.Table(f256[:spec.alphabet], 8)
    assert oracle.unpack(T, P2)[1] == oracle.ERR_CORRUPT
    db = DeviceBatch([to_packed_layer(spec, P2, f256)])
    y = torch.zeros((32, 128), dtype=torch.float32, device="cuda")
    st = torch.cuda.current_stream().cuda_stream
    ans.ans_decode_gemm_bf16(db.h_descs[0][0], x.cuda().data_ptr(), 32, 128, 128, y.data_ptr(), db.status.data_ptr(), st)
    assert db.read_status() != 0
    for M, N, K in ((129, 128, 128), (32, 100, 128), (32, 128, 64)):   # too many rows; N no multiple of 64; N * K != n_symbols
        with pytest.raises(ans.AnsError):
            ans.ans_decode_gemm_bf16(db.h_descs[0][0], x.cuda().data_ptr(), M, N, K, y.data_ptr(), db.status.data_ptr(), st)
