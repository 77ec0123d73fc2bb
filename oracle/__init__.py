"""CPU oracle of the AIF scoring pass: test infrastructure, never imported by the product."""
