"""The C ABI as a C caller sees it: `include/amoeba.h` compiles as C11, the structs that cross the boundary have the
layout the Python binding's ctypes mirrors assume, and a call sequence driven from C gives the values the binding
gives.  The host part needs no GPU; the device part (marked gpu) runs the three data calls from a C program that
uses the CUDA runtime directly and compares what it reads back with the CPU oracle."""
import ctypes as C
import os
import subprocess

import numpy as np
import pytest

import paper_2509_19729_b200 as A
from paper_2509_19729_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HERE = os.path.join(ROOT, "tests", "c_abi")


def _compile(src, out, extra=()):
    lib = str(A.library_path())
    cmd = ["gcc", "-std=c11", "-Wall", "-Werror", "-pedantic", "-I", os.path.join(ROOT, "include"), src, "-o", out,
           lib, f"-Wl,-rpath,{os.path.dirname(lib)}", *extra]
    subprocess.run(cmd, check=True)
    return out


def _kv(text):
    out = {}
    for line in text.splitlines():
        k, _, v = line.partition(" ")
        out[k] = v
    return out


def test_header_is_c11_and_struct_layouts_match_the_binding(tmp_path):
    exe = _compile(os.path.join(HERE, "abi_check.c"), str(tmp_path / "abi_check"))
    got = _kv(subprocess.run([exe], check=True, capture_output=True, text=True).stdout)
    mirrors = {"amoeba_model": B.Model, "amoeba_layout": B.Layout, "amoeba_pad_info": B.PadInfo,
               "amoeba_layer_weights": B.LayerWeights, "amoeba_kv_info": B.KvInfo, "amoeba_weight_desc": B.WeightDesc}
    n_fields = 0
    for cname, cls in mirrors.items():
        assert int(got[f"sizeof.{cname}"]) == C.sizeof(cls), cname
        for field, _ in cls._fields_:
            assert int(got[f"offsetof.{cname}.{field}"]) == getattr(cls, field).offset, (cname, field)
            n_fields += 1
    assert n_fields == sum(1 for k in got if k.startswith("offsetof."))  # every field the C side printed was checked
    # the same plan through the binding gives the same numbers
    m = dict(L=2, hidden=512, Hq=16, Hkv=8, D=128, I=1792)
    plan = A.amoeba_plan_create(A.make_layout(m, 2, 10), A.make_layout(m, 4, 12))
    info = A.amoeba_plan_kv_info(plan)
    assert int(got["plan_create"]) == 0 and int(got["done"]) == 1
    assert int(got["heads_per_run"]) == info.heads_per_run and int(got["run_bytes"]) == info.run_bytes
    assert int(got["src_block_bytes"]) == info.src_block_bytes and int(got["dst_block_bytes"]) == info.dst_block_bytes
    kv, w = A.amoeba_plan_bytes(plan, 3)
    assert int(got["kv_bytes_rw"]) == kv and int(got["w_bytes_rw"]) == w
    assert int(got["workspace_bytes"]) == A.amoeba_rewrite_workspace_bytes(plan, 5, 12)
    assert int(got["dst_pool_bytes"]) == A.amoeba_layout_kv_pool_bytes(A.make_layout(m, 4, 12))
    assert int(got["num_weight_descs"]) == A.amoeba_plan_num_weight_descs(plan)
    assert int(got["desc0_row_bytes"]) == A.amoeba_plan_weight_desc(plan, 0).row_bytes
    assert int(got["set_option"]) == 0 and int(got["bad_option"]) == A.ERR_INVALID_ARG
    assert int(got["null_plan"]) == A.ERR_INVALID_ARG and int(got["unsupported"]) == A.ERR_UNSUPPORTED
    assert got["status_string"] == A.amoeba_status_string(A.ERR_BAD_BLOCK_ID)


CUDA_HOME = os.environ.get("CUDA_HOME", "/usr/local/cuda")


@pytest.mark.gpu
def test_data_calls_driven_from_c_match_the_oracle(tmp_path, oracle):
    """tests/c_abi/abi_e2e.c allocates with cudaMalloc, uploads host-built tables and pools, calls
    amoeba_rewrite_block_tables, amoeba_reshard_kv and amoeba_reshard_weights on a stream of its own, and writes what
    it reads back to a file: compared here byte for byte with the oracle's TP 2 -> 4 result."""
    exe = _compile(os.path.join(HERE, "abi_e2e.c"), str(tmp_path / "abi_e2e"),
                   extra=["-I", os.path.join(CUDA_HOME, "include"), "-L", os.path.join(CUDA_HOME, "lib64"), "-lcudart",
                          f"-Wl,-rpath,{os.path.join(CUDA_HOME, 'lib64')}"])
    m = dict(L=2, hidden=64, Hq=8, Hkv=4, D=32, I=128)
    a, b, T, NB_src, NB_dst = 2, 4, 16, 6, 7
    lens = np.array([40, 0, 17], np.int32)
    g = np.random.default_rng(77)
    nblk = (lens + T - 1) // T
    bt = np.full((3, 3), -1, np.int32)
    ids = g.permutation(NB_src)
    k = 0
    for s, n in enumerate(nblk):
        bt[s, :n] = ids[k:k + n]
        k += int(n)
    free = g.permutation(NB_dst).astype(np.int32)
    KV = g.integers(0, 65536, size=(m["L"], int(nblk.sum()) * T, m["Hkv"], 2, m["D"]), dtype=np.uint16)
    src = oracle.kv_shard(KV, m, T, a, NB_src, lens, bt, fill=0x5A5A)
    W = [{n: g.integers(0, 65536, size=s, dtype=np.uint16) for n, s in oracle.logical_shapes(m).items()}
         for _ in range(m["L"])]
    src_w = [oracle.weights_shard(W[l], m, a) for l in range(m["L"])]
    names = ("q", "o", "gate", "down")  # fused buffers: [q;k;v] under q, [gate;up] under gate
    with open(tmp_path / "in.bin", "wb") as f:
        np.array([m["L"], m["hidden"], m["Hq"], m["Hkv"], m["D"], m["I"], a, b, T, NB_src, NB_dst, 3, 3, len(free)],
                 np.int32).tofile(f)
        lens.tofile(f)
        bt.tofile(f)
        free.tofile(f)
        for p in src:
            p.tofile(f)
        for r in range(a):
            for l in range(m["L"]):
                for n in names:
                    src_w[l][r][n].tofile(f)
    subprocess.run([exe, str(tmp_path / "in.bin"), str(tmp_path / "out.bin")], check=True)
    e_bt, e_pairs, e_n, e_left, e_st = oracle.assign_blocks(lens, T, bt, NB_src, NB_dst, free_list=free)
    e_pools = [np.full(m["L"] * oracle.pool_elems_per_layer(m, T, b, NB_dst), 0xA5A5, np.uint16) for _ in range(b)]
    oracle.kv_transform(m, T, lens, a, NB_src, bt, src, b, NB_dst, e_bt, e_pools)
    e_w = [oracle.weights_transform(src_w[l], m, a, b) for l in range(m["L"])]
    with open(tmp_path / "out.bin", "rb") as f:
        status, n_pairs, left = np.fromfile(f, np.int32, 3)
        assert (status, n_pairs, left) == (e_st, e_n, e_left) and e_st == 0
        assert np.array_equal(np.fromfile(f, np.int32, bt.size).reshape(bt.shape), e_bt)
        for r in range(b):
            assert np.array_equal(np.fromfile(f, np.uint16, e_pools[r].size), e_pools[r]), r
        for r in range(b):
            for l in range(m["L"]):
                for n in names:
                    e = e_w[l][r][n].reshape(-1)
                    assert np.array_equal(np.fromfile(f, np.uint16, e.size), e), (r, l, n)
        assert f.read() == b""
