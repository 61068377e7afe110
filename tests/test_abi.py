"""The C-ABI library loads, exports every symbol include/mdn.h declares, and rejects bad
arguments on the host (no GPU needed: validation happens before any launch)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def mdn():
    from paper_2605_05838_b200 import build
    build.build()
    import paper_2605_05838_b200 as m
    m.lib()
    return m


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "mdn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mdn_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(mdn):
    names = declared_symbols()
    assert "mdn_chunk_fwd" in names and "mdn_chunk_fwd_workspace_bytes" in names and "mdn_status_string" in names
    for n in names:
        assert hasattr(mdn.lib(), n), n


def test_status_strings(mdn):
    assert mdn.status_string(0) == "ok"
    assert all(mdn.status_string(s) for s in range(0, 7))


def params(mdn, **kw):
    base = dict(B=2, T=130, H=3, dk=64, dv=128, chunk=64, num_seqs=0, io_dtype=0, o_dtype=0, path=0, scale=0.125,
                segments=0)
    base.update(kw)
    return mdn.MdnParams(**base)


def test_workspace_layout_and_bounds(mdn):
    p = params(mdn)
    lay = mdn.workspace_layout(p)
    assert lay.num_slots == 2 * 3                      # ceil(130/64) = 3 chunks per row
    assert mdn.workspace_bytes(p) == lay.total_bytes > 0
    assert lay.off_coef % 256 == 0 and lay.off_T % 256 == 0 and lay.off_W % 256 == 0
    assert lay.off_T - lay.off_coef >= lay.num_slots * 3 * mdn.NUM_COEF * 64 * 4
    packed = params(mdn, B=1, T=1000, num_seqs=7)
    assert mdn.workspace_layout(packed).num_slots == 1000 // 64 + 7     # upper bound on sum ceil(len/64)
    assert mdn.host_arena_bytes(p) > mdn.workspace_bytes(p)


def test_host_arena_covers_every_slice_workspace(mdn):
    """mdn_chunk_fwd_host cuts the batch into up to eight slices with B // 8 or B // 8 + 1 rows and calls
    mdn_chunk_fwd on each with its own workspace: the arena's workspace part must cover the LARGEST of the slices'
    needs - a slice with fewer rows can need more (with fewer chains the parallel inter-chunk scan switches on)."""
    up = lambda x: (x + 255) // 256 * 256
    bf = dict(dk=128, dv=128, io_dtype=1, o_dtype=1)
    checked = shrinking = 0
    for B in (1, 2, 7, 8, 9, 15, 17, 33, 40, 64):
        for H in (1, 2, 5, 16):
            for T in (64, 1000, 4096, 16384):
                p = params(mdn, B=B, H=H, T=T, **bf)
                slices = min(B, 8)
                rows, st = B * T * H, H * 128 * 128 * 4
                io = 3 * up(rows * 128 * 2) + 4 * up(rows * 4) + 2 * up(B * st) + up(0) + up(rows * 128 * 2) + 2 * up(B * st)
                ws_part = mdn.host_arena_bytes(p) - io
                need = [mdn.workspace_bytes(params(mdn, B=b, H=H, T=T, **bf)) for b in {B // slices, -(-B // slices)} if b > 0]
                assert ws_part >= slices * up(max(need)), (B, H, T)
                checked += 1
                shrinking += len(need) == 2 and need[0] != need[1] and (need[0] > need[1]) != (B // slices > -(-B // slices))
    assert checked == 160


def test_segment_choice_for_the_parallel_inter_chunk_scan(mdn):
    """Host-side rule only: few long chains are split, anything that already fills the GPU is not."""
    bf = dict(dk=128, dv=128, io_dtype=1, o_dtype=1)
    seg = lambda **kw: mdn.workspace_layout(params(mdn, **{**bf, **kw})).segments
    assert seg(B=1, H=16, T=65536) >= 4              # 16 chains, 1024 chunks each
    assert seg(B=8, H=16, T=4096) == 1               # 128 chains
    assert seg(B=4, H=8, T=2048) == 1                # short
    assert seg(B=1, H=16, T=65536, segments=1) == 1 and seg(B=1, H=16, T=65536, segments=5) == 5
    assert seg(B=1, H=16, T=65536, path=1) == 1      # SIMT path: no scan
    assert seg(B=1, H=16, T=65536, num_seqs=3) == 1  # packed input: no scan
    assert seg(B=1, H=16, T=65536, io_dtype=0, o_dtype=0) == 1
    with_scan = mdn.workspace_layout(params(mdn, **bf, B=1, H=16, T=65536))
    without = mdn.workspace_layout(params(mdn, **bf, B=1, H=16, T=65536, segments=1))
    G = with_scan.segments
    assert with_scan.total_bytes - without.total_bytes >= 16 * ((G - 1) * 2 + (G - 2) * 6) * 128 * 128 * 4
    assert with_scan.off_seg % 256 == 0


@pytest.mark.parametrize("kw", [dict(chunk=32), dict(dk=96), dict(dv=32), dict(B=0), dict(T=0), dict(H=0),
                                dict(io_dtype=5), dict(path=9), dict(num_seqs=3), dict(num_seqs=-1), dict(segments=2),
                                dict(segments=33), dict(segments=-1)])
def test_bad_params_rejected(mdn, kw):
    assert mdn.workspace_bytes(params(mdn, **kw)) == 0


def test_null_and_workspace_errors_before_any_launch(mdn):
    L = mdn.lib()
    p = params(mdn)
    null = ctypes.c_void_p(None)
    fake = ctypes.c_void_p(256 * 4096)   # never dereferenced: rejected by host validation first
    args = [null] * 13
    st = L.mdn_chunk_fwd(ctypes.byref(p), *args, null, 0, null)
    assert mdn.status_string(st).startswith("workspace")
    st = L.mdn_chunk_fwd(ctypes.byref(p), *args, fake, 16, null)
    assert mdn.status_string(st).startswith("workspace")
    st = L.mdn_chunk_fwd(ctypes.byref(p), *args, ctypes.c_void_p(256 * 4096 + 8), 1 << 40, null)
    assert mdn.status_string(st).startswith("workspace")          # misaligned
    st = L.mdn_chunk_fwd(ctypes.byref(p), *args, fake, 1 << 40, null)
    assert mdn.status_string(st) == "invalid argument"            # q is NULL
    bad = params(mdn, chunk=16)
    st = L.mdn_chunk_fwd(ctypes.byref(bad), *args, fake, 1 << 40, null)
    assert mdn.status_string(st).startswith("unsupported")
    # cu_seqlens given but num_seqs == 0
    a2 = list(args); a2[9] = fake
    st = L.mdn_chunk_fwd(ctypes.byref(p), *a2, fake, 1 << 40, null)
    assert mdn.status_string(st) == "invalid argument"


def test_training_buffer_sizes_and_state_image_unpacking(mdn):
    """Host-side arithmetic of the training entry points: per (chunk slot, head) a 64 KB state image and 32 KB of
    fp32 V~ (dR for the adjoint chain, one entry per chunk); and the binding's reading of a state image, checked on a
    hand-built image (value index x key index, two key-index blocks, 16-byte pieces XOR-swizzled with the row)."""
    import numpy as np
    import torch
    L = mdn.lib()
    bf = dict(dk=128, dv=128, io_dtype=1, o_dtype=1)
    p = params(mdn, B=2, T=130, H=3, **bf)                   # 3 chunks per sequence: 6 slots
    per = 3 * (65536 + 64 * 128 * 4)
    assert L.mdn_chunk_states_bytes(ctypes.byref(p)) == 6 * per
    assert L.mdn_bwd_adjoint_states_bytes(ctypes.byref(p)) == 6 * per
    assert L.mdn_chunk_bwd_chunked_workspace_bytes(ctypes.byref(p)) > L.mdn_chunk_bwd_saved_workspace_bytes(ctypes.byref(p)) > 0
    f32 = params(mdn, B=2, T=130, H=3)                      # SIMT path: no chunk-parallel backward
    assert L.mdn_chunk_states_bytes(ctypes.byref(f32)) == 0 and L.mdn_chunk_bwd_chunked_workspace_bytes(ctypes.byref(f32)) == 0

    H, slots = 2, 3
    rng = np.random.default_rng(0)
    S = torch.from_numpy(rng.standard_normal((slots, H, 2, 128, 128)).astype(np.float32)).to(torch.bfloat16)   # [.., S|M, key d, value j]
    img = torch.zeros((slots, H, 2, 2, 128, 64), dtype=torch.bfloat16)        # [.., S|M, key half, row j, 64 keys in swizzled order]
    for j in range(128):
        for piece in range(8):
            for half in range(2):
                src = S[:, :, :, half * 64 + piece * 8: half * 64 + piece * 8 + 8, j]          # logical piece of row j
                phys = piece ^ (j & 7)
                img[:, :, :, half, j, phys * 8: phys * 8 + 8] = src
    vt = torch.from_numpy(rng.standard_normal((slots, 64, H, 128)).astype(np.float32))
    buf = torch.cat([img.view(torch.uint8).reshape(-1), vt.view(torch.uint8).reshape(-1)])
    assert buf.numel() == slots * H * (65536 + 32768)
    Sg, Mg = mdn.unpack_chunk_states(buf, H)
    assert torch.equal(Sg, S[:, :, 0].float()) and torch.equal(Mg, S[:, :, 1].float())
    assert torch.equal(mdn.unpack_chunk_vt(buf, H), vt)
    with pytest.raises(ValueError):
        mdn.unpack_chunk_states(buf[:-4], H)
