"""The header is consumed by a C99 compiler and the library is called from C
(host-only entry points; no GPU needed)."""
import os
import shutil
import subprocess

import pytest

from paper_2408_08147_b200 import build as pdkv_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_header_is_plain_c_and_callable_from_c(tmp_path):
    gcc = shutil.which("gcc")
    if gcc is None:
        pytest.skip("no gcc")
    lib = pdkv_build.build_library()
    exe = str(tmp_path / "host_only")
    subprocess.check_call([gcc, "-std=c99", "-pedantic", "-Wall", "-Wextra", "-Werror",
                           "-I", os.path.join(ROOT, "include"),
                           os.path.join(ROOT, "tests", "c_abi", "host_only.c"),
                           "-o", exe, lib, "-Wl,-rpath," + os.path.dirname(lib)])
    out = subprocess.run([exe], capture_output=True, text=True, timeout=120)
    assert out.returncode == 0, out.stdout + out.stderr
    got = dict(line.split(" ", 1) for line in out.stdout.strip().splitlines())
    # geometry: L=2, H=2, D=16, E=2 -> one token is 2*L*H*D*E = 256 bytes, one head row 32 bytes
    tok = 2 * 2 * 2 * 16 * 2
    assert int(got["pool_bytes_src"]) == 6 * 4 * tok
    assert int(got["pool_bytes_dst"]) == 4 * 8 * tok
    assert got["strerror_ok"] == "ok"
    assert int(got["tile_bytes"]) == 32768
    assert int(got["buffer_bytes"]) == (5 + 9) * tok
    assert [int(x) for x in got["req_off"].split()] == [0, 5 * tok, 14 * tok]
    # fused traffic: payload read; payload + zero padding written (3 + 7 empty slots of the two last decode blocks)
    assert [int(x) for x in got["traffic"].split()] == [14 * tok, (14 + 3 + 7) * tok]
    # pack tiles never cross a 4-token prefill block: 5 tokens -> 2 tiles, 9 tokens -> 3 tiles
    f = got["pack_tiles"].split()
    assert int(f[0]) == 5
    # first tile: prefill block 3, slot 0 (block-major: block * 2*L*B*H*D*E), buffer offset 0, 4 tokens
    assert int(f[2]) == 3 * (2 * 2 * 4 * 2 * 16 * 2) and int(f[4]) == 0 and int(f[6]) == 4
    assert int(got["pack_launches"]) == 1
    # 32-byte rows, tiny tiles: groups of threads in a 512-thread CTA, 32-byte accesses, register copy;
    # the plan kept "ctas_per_sm" = 0 (automatic: 2 here) although the tunable was 7 when it was asked
    assert [int(x) for x in got["launch_shape"].split()] == [512, 32, 2, 0, 0]
    assert int(got["transfer_on_dry_plan"]) == -1          # PDKV_ERR_INVALID_ARG
    assert int(got["duplicate_decode_block"]) == -3        # PDKV_ERR_TABLE
