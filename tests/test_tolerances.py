"""What the attention tolerance rests on (CPU only).

The stated bound for bf16 attention outputs is 2e-2 max-abs.  An output is STORED in bf16; for a value of
magnitude 4 or more the storage rounding alone can cost 2^-6 = 0.0156, which the oracle (unrounded float64) does
not have.  tests.parity.attention_bound therefore allows the larger of 2e-2 and (half a bf16 spacing of the value
plus 2^-8 of it); the second is the larger from magnitude 3.12 on."""
import numpy as np

from oracle import quoka_oracle as O
from tests.parity import attention_bound


def test_bound_is_the_stated_one_up_to_magnitude_3():
    x = np.linspace(-3.12, 3.12, 4001)
    assert (attention_bound(x, "bf16") == 2e-2).all()
    # between 3.12 and 4: half a spacing of 2^-6 plus 2^-8 |o|, at most 0.0235
    y = np.linspace(3.13, 3.999, 100)
    b = attention_bound(y, "bf16")
    np.testing.assert_allclose(b, 2.0 ** -7 + y * 2.0 ** -8)
    assert (b > 2e-2).all() and (b < 0.0235).all()
    assert (attention_bound(np.array([0.0, 5.0, -100.0]), "f32") == 2e-4).all()


def test_storage_rounding_alone_reaches_half_a_spacing():
    # midpoints between neighbouring bf16 values in [4, 8): rounding moves them by exactly 2^-6
    x = 4.0 + 2.0 ** -5 * (np.arange(100) + 0.5)
    err = np.abs(O.round_to_bf16(x) - x)
    assert np.allclose(err, 2.0 ** -6)
    # which leaves the arithmetic less than a quarter of the stated 2e-2
    assert 2e-2 - 2.0 ** -6 < 0.005
    b = attention_bound(x, "bf16")
    assert (b > 2.0 ** -6).all() and (b <= 2.0 ** -6 + 8 * 2.0 ** -8).all()


def test_bound_grows_with_the_spacing_of_the_stored_value():
    for lo in (4.0, 8.0, 16.0, 64.0):
        spacing = lo * 2.0 ** -7
        x = np.array([lo, lo * 1.5, np.nextafter(2 * lo, 0)])
        np.testing.assert_allclose(attention_bound(x, "bf16"), spacing / 2 + x * 2.0 ** -8)
        np.testing.assert_allclose(attention_bound(-x, "bf16"), spacing / 2 + x * 2.0 ** -8)
