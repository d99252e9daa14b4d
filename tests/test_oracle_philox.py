"""Pins for the oracle's counter-based generator (Philox4x32-10, Salmon et al., SC'11).

The generator is not part of the paper; it stands in for real gradients.  It is pinned against
(a) a library implementation of the same published generator (Triton's `philox_impl`, run on the
CPU through Triton's interpreter), (b) NumPy's Philox4x64 through a width-generic restatement that
must match NumPy at 64 bits and the oracle at 32 bits, and (c) avalanche / uniformity properties.
"""
import os
import subprocess
import sys
import textwrap

import numpy as np
import pytest

M32 = (0xD2511F53, 0xCD9E8D57, 0x9E3779B9, 0xBB67AE85)
M64 = (0xD2E7470EE14C6C93, 0xCA5A826395121157, 0x9E3779B97F4A7C15, 0xBB67AE8584CAA73B)


def philox_generic(ctr, key, width, consts, rounds=10):
    mask = (1 << width) - 1
    m0, m1, w0, w1 = consts
    c = list(ctr)
    k = list(key)
    for r in range(rounds):
        if r:
            k = [(k[0] + w0) & mask, (k[1] + w1) & mask]
        p0, p1 = m0 * c[0], m1 * c[2]
        c = [(p1 >> width) ^ c[1] ^ k[0], p1 & mask, (p0 >> width) ^ c[3] ^ k[1], p0 & mask]
    return c


def test_generic_restatement_matches_numpy_philox4x64():
    rng = np.random.default_rng(11)
    for _ in range(20):
        ctr = [int(x) for x in rng.integers(0, 2**63, 4, dtype=np.uint64)]
        key = [int(x) for x in rng.integers(0, 2**63, 2, dtype=np.uint64)]
        bg = np.random.Philox(counter=np.array(ctr, dtype=np.uint64), key=np.array(key, dtype=np.uint64))
        got = [int(x) for x in bg.random_raw(4)]
        nxt = list(ctr)
        nxt[0] += 1  # NumPy advances the counter before producing a block
        assert got == philox_generic(nxt, key, 64, M64)


def test_oracle_matches_generic_restatement_at_32_bits(oracle):
    rng = np.random.default_rng(12)
    for _ in range(200):
        ctr = [int(x) for x in rng.integers(0, 2**32, 4, dtype=np.uint64)]
        key = [int(x) for x in rng.integers(0, 2**32, 2, dtype=np.uint64)]
        assert [int(x) for x in oracle.philox4x32_10(ctr, key)] == philox_generic(ctr, key, 32, M32)


TRITON_SNIPPET = textwrap.dedent("""
    import os, sys
    os.environ["TRITON_INTERPRET"] = "1"
    import numpy as np, torch, triton, triton.language as tl

    @triton.jit
    def kern(cp, kp, op, BLOCK: tl.constexpr):
        offs = tl.arange(0, BLOCK)
        c0 = tl.load(cp + 4 * offs + 0).to(tl.uint32, bitcast=True)
        c1 = tl.load(cp + 4 * offs + 1).to(tl.uint32, bitcast=True)
        c2 = tl.load(cp + 4 * offs + 2).to(tl.uint32, bitcast=True)
        c3 = tl.load(cp + 4 * offs + 3).to(tl.uint32, bitcast=True)
        k0 = tl.load(kp + 2 * offs + 0).to(tl.uint32, bitcast=True)
        k1 = tl.load(kp + 2 * offs + 1).to(tl.uint32, bitcast=True)
        r0, r1, r2, r3 = tl.random.philox_impl(c0, c1, c2, c3, k0, k1, 10)
        tl.store(op + 4 * offs + 0, r0.to(tl.int32, bitcast=True))
        tl.store(op + 4 * offs + 1, r1.to(tl.int32, bitcast=True))
        tl.store(op + 4 * offs + 2, r2.to(tl.int32, bitcast=True))
        tl.store(op + 4 * offs + 3, r3.to(tl.int32, bitcast=True))

    n = 64
    rng = np.random.default_rng(2111)
    ctr = rng.integers(0, 2**32, (n, 4), dtype=np.uint64).astype(np.uint32)
    key = rng.integers(0, 2**32, (n, 2), dtype=np.uint64).astype(np.uint32)
    ctr[0] = 0; key[0] = 0
    ctr[1] = 0xFFFFFFFF; key[1] = 0xFFFFFFFF
    out = torch.zeros(n * 4, dtype=torch.int32)
    kern[(1,)](torch.from_numpy(ctr.view(np.int32).reshape(-1).copy()),
               torch.from_numpy(key.view(np.int32).reshape(-1).copy()), out, BLOCK=n)
    np.save(sys.argv[1], np.stack([ctr.reshape(-1)[: n * 4].astype(np.uint32),
                                   np.pad(key.reshape(-1), (0, n * 2)).astype(np.uint32),
                                   out.numpy().view(np.uint32)]))
""")


def test_oracle_matches_library_philox(oracle, tmp_path):
    pytest.importorskip("triton")
    script = tmp_path / "tp.py"
    script.write_text(TRITON_SNIPPET)
    res = tmp_path / "out.npy"
    env = dict(os.environ, TRITON_INTERPRET="1", CUDA_VISIBLE_DEVICES="")
    p = subprocess.run([sys.executable, str(script), str(res)], env=env, capture_output=True,
                       text=True, timeout=600)
    if p.returncode != 0:
        pytest.skip("Triton's CPU interpreter is not usable here: " + p.stderr[-300:])
    data = np.load(res)
    n = 64
    ctr = data[0].reshape(n, 4)
    key = data[1][: 2 * n].reshape(n, 2)
    lib_words = data[2].reshape(n, 4)
    for i in range(n):
        assert np.array_equal(oracle.philox4x32_10(ctr[i], key[i]), lib_words[i]), i


def test_avalanche(oracle):
    """Flipping any single counter or key bit flips about half of the 128 output bits."""
    base_c = np.array([0x243F6A88 & 0xFFFFFFFF, 17, 3, 0x47000000], dtype=np.uint32)
    base_k = np.array([0x48414446, 0], dtype=np.uint32)
    ref = oracle.philox4x32_10(base_c, base_k)
    flips = []
    for word in range(6):
        for bit in range(32):
            c, k = base_c.copy(), base_k.copy()
            if word < 4:
                c[word] ^= np.uint32(1 << bit)
            else:
                k[word - 4] ^= np.uint32(1 << bit)
            out = oracle.philox4x32_10(c, k)
            d = sum(bin(int(a) ^ int(b)).count("1") for a, b in zip(out, ref))
            flips.append(d)
    flips = np.array(flips)
    assert flips.min() >= 35 and flips.max() <= 93     # 64 +- 5 sigma (sigma = sqrt(32) = 5.7)
    assert abs(flips.mean() - 64.0) < 2.0


def test_words_are_uniform(oracle):
    n = 20000
    ctrs = np.zeros((n, 4), dtype=np.uint32)
    ctrs[:, 0] = np.arange(n)
    ctrs[:, 3] = 0x47000000
    words = oracle.philox4x32_10_many(ctrs, [123, 456]).reshape(-1)
    counts = np.bincount(words.view(np.uint8), minlength=256).astype(np.float64)
    expected = words.size * 4 / 256.0
    chi2 = ((counts - expected) ** 2 / expected).sum()
    assert chi2 < 255 + 5 * np.sqrt(2 * 255)          # 5 sigma
    # distinct counters give distinct blocks (the round function is a bijection of the counter)
    assert len({tuple(r) for r in words.reshape(n, 4)}) == n


def test_stream_separation(oracle):
    """Gradient, initial-model and selection streams never share a counter: their outputs differ."""
    g = oracle.grad_normals(9, 5, 0, 0)
    i = oracle.init_normals(9, 5)
    assert not np.array_equal(g, i)
    assert oracle.select_bits(9, 0, 5) != oracle.select_bits(9, 5, 0)
    # device, step and group each select a different block
    assert not np.array_equal(oracle.grad_normals(9, 5, 1, 0), oracle.grad_normals(9, 5, 0, 1))
    assert not np.array_equal(oracle.grad_normals(9, 5, 1, 0), oracle.grad_normals(9, 6, 1, 0))
    # 2^32 steps later is a different block, not a wrap-around
    assert not np.array_equal(oracle.grad_normals(9, 5, 1, 0), oracle.grad_normals(9, 5, 1 + 2**32, 0))
