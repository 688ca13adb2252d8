"""The shared library builds, loads without a GPU, and exports every entry point the header
declares.  Only host-side helpers are called here (no kernels)."""
import ctypes
import os
import re

from paper_2509_08721_b200 import binding as B
from paper_2509_08721_b200 import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "sapo.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sapo_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_entry_point():
    path = build.build()
    lib = ctypes.CDLL(path)
    names = declared_functions()
    assert set(B.EXPORTS) <= set(names)
    assert {"sapo_pack_rollouts", "sapo_group_advantages", "sapo_policy_loss_fwd",
            "sapo_policy_loss_bwd"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_host_side_helpers():
    lib = B.load()
    assert lib.sapo_status_string(0) == b"ok"
    assert b"workspace" in lib.sapo_status_string(-3)
    # forward scratch: three partial arrays per vocab split; backward: a bf16 dz panel
    T, H, V = 18432, 896, 151936
    fwd = B.sapo_workspace_bytes(B.WS_FWD, T, H, V, B.DTYPE_BF16)
    assert fwd >= 3 * 4 * T and fwd % 256 == 0
    bwd = B.sapo_workspace_bytes(B.WS_BWD, T, H, V, B.DTYPE_BF16)
    k_split_scratch = 3 * 96 * 256 * 512 * 4              # partial accumulator tiles of K-split parts
    assert bwd == T * V * 2 + k_split_scratch            # V is already a multiple of 128
    assert B.sapo_workspace_bytes_min(B.WS_BWD, T, H, V, B.DTYPE_BF16) == 128 * V * 2 + k_split_scratch
    # single-pass call: the panel plus, per token, a scaled hidden row and a few floats
    fused = B.sapo_workspace_bytes(B.WS_FUSED, T, H, V, B.DTYPE_BF16)
    assert T * (V + H) * 2 + k_split_scratch < fused < T * (V + H) * 2 + k_split_scratch + 3000 * T
    assert 0 < B.sapo_workspace_bytes_min(B.WS_FUSED, T, H, V, B.DTYPE_BF16) < fused // 10
    assert B.sapo_workspace_bytes(B.WS_FUSED, T, H, V, B.DTYPE_F32) == 0       # bf16 operands only
    assert B.sapo_workspace_bytes(B.WS_FWD, T, 12, V, B.DTYPE_BF16) == 0      # H % 8 != 0
    assert B.sapo_workspace_bytes(7, T, H, V, B.DTYPE_BF16) == 0
    f32 = B.sapo_workspace_bytes(B.WS_FWD, 1024, 64, 1000, B.DTYPE_F32)
    assert f32 >= (1024 + 1000) * 3 * 64 * 2
    assert B.decode_status(0x21) == ["TOKEN_OVERFLOW", "WAIT_TIMEOUT"]


def test_header_is_plain_c(tmp_path):
    """include/sapo.h is the boundary: it must compile as C99 on its own (no C++, no CUDA or
    torch types), and every status / error code it defines must have a text."""
    import subprocess
    src = tmp_path / "use_header.c"
    src.write_text('#include "sapo.h"\n'
                   "int main(void) { sapo_loss_cfg c; c.eps_low = 0.2f; (void)c;\n"
                   "  return sizeof(sapo_packed) > 0 && SAPO_WS_FUSED == 3 ? 0 : 1; }\n")
    inc = os.path.join(ROOT, "include")
    res = subprocess.run(["gcc", "-std=c99", "-Wall", "-Werror", "-pedantic", "-fsyntax-only", "-I", inc, str(src)],
                         capture_output=True, text=True)
    assert res.returncode == 0, res.stderr
    lib = B.load()
    for code in range(0, -6, -1):
        assert lib.sapo_status_string(code) != b"unknown code"


def test_pack_rejects_null_arrays_on_the_host():
    """A NULL array the sizes say will be touched is an argument error, found before any launch
    (so this needs no GPU): it must not become a fault on the device."""
    import ctypes as C
    lib = B.load()
    x = 0x1000                                  # any non-NULL value: nothing dereferences it on the host
    def bufs(**kw):
        full = dict(hidden=x, ids=x, old_logp=x, offsets=x, rewards=x, n_rollouts=4)
        full.update(kw)
        return B.RolloutBufC(*[full[k] for k in ("hidden", "ids", "old_logp", "offsets", "rewards", "n_rollouts")])
    sel = B.SelectionC(x, x, x, x, 2)
    def packed(**kw):
        names = ("hidden", "ids", "old_logp", "rewards", "cu_seqlens", "seq_group", "seq_is_ext", "seq_src",
                 "tok_seq", "tok_mask", "group_offsets", "n_tokens", "n_seqs")
        full = {k: x for k in names}
        full.update(kw)
        return B.PackedC(*[full[k] for k in names], 128, 8)
    def call(local, ext, out, selection=sel):
        return lib.sapo_pack_rollouts(C.byref(local), C.byref(ext), C.byref(selection), 64, B.DTYPE_BF16,
                                      C.byref(out), x, None)
    for member in ("hidden", "ids", "old_logp", "offsets", "rewards"):
        assert call(bufs(**{member: None}), bufs(), packed()) == -1, member
        assert call(bufs(), bufs(**{member: None}), packed()) == -1, member
    for member in ("hidden", "ids", "old_logp", "rewards", "cu_seqlens", "seq_group", "seq_is_ext", "seq_src",
                   "tok_seq", "tok_mask", "group_offsets", "n_tokens", "n_seqs"):
        assert call(bufs(), bufs(), packed(**{member: None})) == -1, member
    assert call(bufs(), bufs(), packed(), B.SelectionC(None, x, x, x, 2)) == -1
    assert call(bufs(), bufs(), packed(), B.SelectionC(x, x, None, x, 2)) == -1


def test_default_panel_size_fills_the_last_wave_of_the_dhidden_contraction():
    """Batches beyond 20 480 tokens are cut into equal chunks whose count the workspace query
    picks so that the dhidden contraction (2, 3 or 7 column tiles per 256-token block at H = 896,
    1536, 3584; 74 CTA pairs) wastes least of its last wave.  The chunk rows follow from the size
    of the dz panel, the only per-row part of the separate backward's scratch."""
    def panel_rows(T, H, V):
        full = B.sapo_workspace_bytes(B.WS_BWD, T, H, V, B.DTYPE_BF16)
        least = B.sapo_workspace_bytes_min(B.WS_BWD, T, H, V, B.DTYPE_BF16)
        vp = -(-V // 128) * 128
        assert (full - least) % (2 * vp) == 0
        return (full - least) // (2 * vp) + 128
    assert panel_rows(16527, 896, 151936) == 16640            # up to 20 480 tokens: the whole batch
    assert panel_rows(20480, 896, 151936) == 20480
    # 332 751 tokens at H = 896: 18 chunks of 18 560 (146 tiles = two full waves), not 17 of 19 584
    assert panel_rows(332751, 896, 151936) == 18560
    # H = 1536 and 3584: chunks of at most 16 384 tokens (a chunk's hidden rows stay within 48 MB)
    assert panel_rows(146382, 1536, 151936) == 13312          # 11 chunks; 9 of 16 384 waste a third of a wave
    assert panel_rows(143347, 3584, 152064) == 14336          # 10 chunks
    for T, H, V in ((146382, 1536, 151936), (143347, 3584, 152064), (332751, 896, 151936), (50000, 256, 4096)):
        rows = panel_rows(T, H, V)
        assert rows % 128 == 0 and 128 <= rows <= 20480
        n = -(-T // rows)
        assert (n - 1) * rows < T <= n * rows and n * rows - T < n * 128   # equal chunks, no short one at the end
