"""Host-side checks of the seeded input generators (no method arithmetic lives there)."""
import numpy as np

from paper_2602_11812_b200 import inputs as gen


def test_bf16_rounding_is_nearest_even_and_exact():
    x = np.array([1.0, 1.00390625, 1.0 + 2**-8, 1.0 + 3 * 2**-8, -2.7182817, 3.0e38, 1e-40], dtype=np.float32)
    r = gen.round_to_bf16(x)
    bits = gen.bf16_bits(r)
    assert r[0] == 1.0 and r[1] == 1.0 and r[2] == 1.0            # ties go to the even mantissa
    assert r[3] == np.float32(1.0 + 2**-6)                        # 1 + 3/256 is a tie between 1+2/256 and 1+4/256 -> even
    back = (bits.astype(np.uint32) << 16).view(np.float32)
    assert np.array_equal(back, r)
    assert np.all(np.abs(r[:5] - x[:5]) <= np.abs(x[:5]) * 2.0**-8)


def test_named_configs_have_the_stated_shapes():
    c1 = gen.config_tiny()
    assert c1.lengths.tolist() == [16, 31, 48, 64] and c1.T == 159 and c1.d == 256 and c1.V == 4096
    assert c1.head.m_h == 128 and c1.head.d_out == 1 and c1.dtype == "f32"
    assert abs(float(c1.W.std()) - 1 / 16) < 2e-3 and abs(float(c1.hidden.std()) - 1.0) < 2e-2
    c1b = gen.config_tiny(gen.HEAD_BINS)
    assert c1b.head.d_out == 20 and abs(c1b.head.centres[0] - 204.8) < 1e-3
    assert np.array_equal(c1b.hidden, c1.hidden) and np.array_equal(c1b.W, c1.W)
    c2 = gen.config_mid(V=512, d=256, m_h=64)
    assert c2.B == 32 and c2.lengths.min() >= 32 and c2.lengths.max() <= 2048
    assert c2.T == 9555                                           # the seed-1 draw of lognormal(5.5, 0.8)
    assert np.all(gen.bf16_bits(c2.hidden) >= 0)                  # raises if a value is not bf16-exact
    ch_rms = np.sqrt((c2.hidden.astype(np.float64) ** 2).mean(axis=0))
    assert int((ch_rms > 10).sum()) == 3                          # 1 % of 256 channels, gain 20
    c3 = gen.config_long(V=256, d=64, m_h=32)
    assert c3.B == 64 and c3.lengths.min() >= 128 and c3.lengths.max() <= 8192 and c3.offsets.dtype == np.int32
    assert c3.T == int(c3.lengths.sum()) == int(c3.offsets[-1])


def test_retire_schedule_keeps_every_slot_live():
    reset, drawn = gen.retire_schedule(7, steps=200, slots=16, mu=3.0, sigma=1.0)
    assert reset.shape == (200, 16) and np.all(reset[0] == gen.RESET_EMPTY)
    assert set(np.unique(reset)) <= {gen.RESET_KEEP, gen.RESET_EMPTY}
    assert (reset[1:] == gen.RESET_EMPTY).sum() > 16              # sequences retire and are replaced
    assert len(drawn) == (reset == gen.RESET_EMPTY).sum()
    p = gen.config_rl_group(prompts=3, group=4, steps=5, d=64, V=128, m_h=16, min_len=4, max_len=9)
    assert p.slots == 12 and p.reset_src[0].tolist() == [0] * 4 + [1] * 4 + [2] * 4
    assert np.all(p.reset_src[1:] == gen.RESET_KEEP) and p.prompts.B == 3
