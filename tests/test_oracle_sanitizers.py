"""The C oracle and the host-only library parts under AddressSanitizer and UBSan (no GPU needed)."""
import os
import shutil
import subprocess

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.skipif(shutil.which("gcc") is None, reason="needs gcc")
def test_oracle_is_clean_under_asan_and_ubsan(tmp_path):
    exe = str(tmp_path / "oracle_san")
    build = subprocess.run(
        ["gcc", "-O1", "-g", "-std=c11", "-fsanitize=address,undefined", "-fno-sanitize-recover=all",
         os.path.join(ROOT, "oracle", "kvc_oracle.c"),
         os.path.join(ROOT, "tests", "native", "oracle_sanitizer_driver.c"), "-o", exe],
        capture_output=True, text=True)
    if build.returncode != 0 and "sanitize" in build.stderr:
        pytest.skip("sanitizer runtime not installed")
    assert build.returncode == 0, build.stderr
    run = subprocess.run([exe], capture_output=True, text=True, timeout=120)
    assert run.returncode == 0 and run.stdout.strip() == "ok", run.stdout + run.stderr


@pytest.mark.skipif(shutil.which("g++") is None, reason="needs g++")
def test_host_only_library_parts_are_clean_under_asan_and_ubsan(tmp_path):
    """The slot policy and the chunk-file store have no CUDA dependency: build them straight from
    their sources with the sanitizers and run a driver over their entry points."""
    csrc = os.path.join(ROOT, "paper_2609_11744_b200", "csrc")
    exe = str(tmp_path / "host_san")
    build = subprocess.run(
        ["g++", "-O1", "-g", "-std=c++17", "-fsanitize=address,undefined", "-fno-sanitize-recover=all",
         "-I", os.path.join(ROOT, "include"), os.path.join(csrc, "kvc_slot_pool.cpp"),
         os.path.join(csrc, "kvc_store.cpp"),
         os.path.join(ROOT, "tests", "native", "host_sanitizer_driver.cpp"), "-o", exe, "-lpthread"],
        capture_output=True, text=True)
    if build.returncode != 0 and "sanitize" in build.stderr:
        pytest.skip("sanitizer runtime not installed")
    assert build.returncode == 0, build.stderr
    scratch = tmp_path / "store"
    scratch.mkdir()
    run = subprocess.run([exe, str(scratch)], capture_output=True, text=True, timeout=120)
    assert run.returncode == 0 and run.stdout.strip() == "ok", run.stdout + run.stderr


@pytest.mark.skipif(shutil.which("g++") is None, reason="needs g++")
def test_staging_ring_is_clean_under_asan_and_ubsan(tmp_path):
    """The ring's bookkeeping, FIFO and pool mode, compiled as plain C++ (the CUDA runtime calls it
    names are stubbed in the driver and never reached) and driven by a long random walk."""
    cuda_inc = os.path.join(os.environ.get("CUDA_HOME", "/usr/local/cuda"), "include")
    if not os.path.isdir(cuda_inc):
        pytest.skip("needs the CUDA toolkit headers")
    csrc = os.path.join(ROOT, "paper_2609_11744_b200", "csrc")
    exe = str(tmp_path / "ring_san")
    build = subprocess.run(
        ["g++", "-O1", "-g", "-std=c++17", "-fsanitize=address,undefined", "-fno-sanitize-recover=all",
         "-I", os.path.join(ROOT, "include"), "-I", csrc, "-I", cuda_inc,
         "-x", "c++", os.path.join(csrc, "kvc_ring.cu"), os.path.join(csrc, "kvc_slot_pool.cpp"),
         os.path.join(ROOT, "tests", "native", "ring_sanitizer_driver.cpp"), "-o", exe, "-lpthread"],
        capture_output=True, text=True)
    if build.returncode != 0 and "sanitize" in build.stderr:
        pytest.skip("sanitizer runtime not installed")
    assert build.returncode == 0, build.stderr
    run = subprocess.run([exe], capture_output=True, text=True, timeout=120)
    assert run.returncode == 0 and run.stdout.strip() == "ok", run.stdout + run.stderr


@pytest.mark.skipif(shutil.which("g++") is None, reason="needs g++")
def test_layout_mapper_and_launch_front_ends_are_clean_under_asan_and_ubsan(tmp_path):
    """kvc_layout.cu compiled as plain C++ with host stand-ins for the CUDA runtime and a launch
    recorder instead of the kernels: validation, the chunk mapper, the shared-prefix trie and the
    per-block tables over 200 random geometries, tunings and request sets."""
    cuda_inc = os.path.join(os.environ.get("CUDA_HOME", "/usr/local/cuda"), "include")
    if not os.path.isdir(cuda_inc):
        pytest.skip("needs the CUDA toolkit headers")
    csrc = os.path.join(ROOT, "paper_2609_11744_b200", "csrc")
    exe = str(tmp_path / "layout_san")
    build = subprocess.run(
        ["g++", "-O1", "-g", "-std=c++17", "-fsanitize=address,undefined", "-fno-sanitize-recover=all",
         "-I", os.path.join(ROOT, "include"), "-I", csrc, "-I", cuda_inc,
         "-x", "c++", os.path.join(csrc, "kvc_layout.cu"),
         os.path.join(ROOT, "tests", "native", "layout_sanitizer_driver.cpp"), "-o", exe, "-lpthread"],
        capture_output=True, text=True)
    if build.returncode != 0 and "sanitize" in build.stderr:
        pytest.skip("sanitizer runtime not installed")
    assert build.returncode == 0, build.stderr
    run = subprocess.run([exe], capture_output=True, text=True, timeout=300)
    assert run.returncode == 0 and run.stdout.strip() == "ok", run.stdout + run.stderr[-3000:]


@pytest.mark.skipif(shutil.which("g++") is None, reason="needs g++")
def test_host_transfers_move_whole_requests_on_the_host_under_asan_and_ubsan(tmp_path):
    """kvc_offload_to_host / kvc_load_from_host with the library's host code compiled as plain C++, the
    CUDA runtime replaced by host stand-ins and the kernel launch by a loop over the slabs the launch
    names: 120 random geometries, ring sizes and kinds; host images and pools checked byte for byte,
    every buffer exactly as large as the interface requires."""
    cuda_inc = os.path.join(os.environ.get("CUDA_HOME", "/usr/local/cuda"), "include")
    if not os.path.isdir(cuda_inc):
        pytest.skip("needs the CUDA toolkit headers")
    csrc = os.path.join(ROOT, "paper_2609_11744_b200", "csrc")
    exe = str(tmp_path / "host_transfer_san")
    build = subprocess.run(
        ["g++", "-O1", "-g", "-std=c++17", "-fsanitize=address,undefined", "-fno-sanitize-recover=all",
         "-I", os.path.join(ROOT, "include"), "-I", csrc, "-I", cuda_inc,
         "-x", "c++", os.path.join(csrc, "kvc_layout.cu"), os.path.join(csrc, "kvc_ring.cu"),
         os.path.join(csrc, "kvc_slot_pool.cpp"), os.path.join(csrc, "kvc_host_transfer.cpp"),
         os.path.join(ROOT, "tests", "native", "host_transfer_sanitizer_driver.cpp"), "-o", exe, "-lpthread"],
        capture_output=True, text=True)
    if build.returncode != 0 and "sanitize" in build.stderr:
        pytest.skip("sanitizer runtime not installed")
    assert build.returncode == 0, build.stderr
    run = subprocess.run([exe], capture_output=True, text=True, timeout=300)
    assert run.returncode == 0 and run.stdout.strip() == "ok", run.stdout + run.stderr[-3000:]
